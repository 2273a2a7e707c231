"""firp_topb_static -- the entry point that allocates nothing -- against firp_step.

Some hosts of this library may not allocate device memory while decoding (a serving loop with a
memory pool fixed at start-up, a plug-in that only ever receives buffers from its host), so this
one call keeps its scratch in a fixed array inside the library.  Here it is run, through the C ABI,
on the logits that firp_step exported, twice in a row on different logits, and must reproduce the
selections firp_step made from the same rows: the greedy token of every tree row and the ordered
top-B ids and values of every pseudo row, exactly (both paths select from the same fp32 numbers).
The file name sorts last on purpose: a run that stops at the first failure has by then run every
other test.
"""
import numpy as np
import pytest

import synth_inputs as si

pytestmark = pytest.mark.gpu


def test_static_topb_matches_step_twice_in_a_row(c1, c1_weights):
    import torch
    assert torch.cuda.is_available(), "this test needs a CUDA device"
    from paper_2410_20488_b200 import FirpEngine, FirpError, binding, build as firp_build, firp_topb_static
    firp_build.build()
    parents = si.tree_template(c1.T)
    eng = FirpEngine(c1, c1_weights, max_ctx=256)
    T, k, V, B = c1.T, c1.k, c1.V, eng.B
    d_prompt = torch.from_numpy(si.prompt(c1)).cuda()
    pout = eng.new_out(1, 1, k, T_next=T)
    eng.prefill(0, d_prompt, k, c1.l, parents, pout)
    out = eng.new_out(1, T, k)
    ids = torch.full((T + k, B), -1, dtype=torch.int32, device="cuda")
    vals = torch.zeros((T + k, B), dtype=torch.float32, device="cuda")
    tokens = pout.next_tree_tokens[0].clone()
    for call in range(2):                     # two calls in a row share the built-in scratch
        eng.step(tokens, parents, k, c1.l, out)
        ids.fill_(-1)
        firp_topb_static(out.logits.data_ptr(), T + k, V, B, ids.data_ptr(), vals.data_ptr(), eng.stream)
        torch.cuda.synchronize()
        got_ids, got_vals = ids.cpu().numpy(), vals.cpu().numpy()
        assert np.array_equal(got_ids[:T, 0], out.best[0].cpu().numpy()), "greedy tokens differ (call %d)" % call
        assert np.array_equal(got_ids[T:], out.topb_ids[0, :k].cpu().numpy()), "top-B ids differ (call %d)" % call
        assert np.array_equal(got_vals[T:], out.topb_vals[0, :k].cpu().numpy()), "top-B values differ (call %d)" % call
        logits = out.logits[0].cpu().numpy()
        want = np.stack([np.lexsort((np.arange(V), -row))[:B] for row in logits])
        assert np.array_equal(got_ids, want), "not the top-B of the logits (call %d)" % call
        eng.commit(1)
        tokens = out.next_tree_tokens[0].clone()
    # sizes beyond the built-in scratch are refused, not truncated
    with pytest.raises(FirpError) as e:
        firp_topb_static(out.logits.data_ptr(), 4097, V, B, ids.data_ptr(), vals.data_ptr(), eng.stream)
    assert e.value.code == binding.FIRP_ERR_CAPACITY
    with pytest.raises(FirpError) as e:
        firp_topb_static(out.logits.data_ptr(), T + k, V, 9, ids.data_ptr(), vals.data_ptr(), eng.stream)
    assert e.value.code == binding.FIRP_ERR_BAD_ARG
    eng.close()


@pytest.mark.parametrize("rows,vocab,b", [(1365, 5000, 5), (256, 32000, 3), (2, 4097, 8), (4096, 2048, 1), (7, 1, 1)])
def test_static_topb_many_segments_and_ragged_tails(rows, vocab, b):
    """The same call on synthetic fp32 logits whose rows span several 2048-logit segments with a ragged last
    one, at row counts that fill the built-in scratch almost to its 4096 slots (1365 x 3 = 4095, 256 x 16 =
    4096), with b < 8, and with planted ties; twice in a row on different data."""
    import torch
    assert torch.cuda.is_available(), "this test needs a CUDA device"
    from paper_2410_20488_b200 import FirpError, binding, build as firp_build, firp_topb_static
    firp_build.build()
    stream = torch.cuda.current_stream().cuda_stream
    ids = torch.empty((rows, b), dtype=torch.int32, device="cuda")
    vals = torch.empty((rows, b), dtype=torch.float32, device="cuda")
    for call in range(2):
        bits = si.normal_bf16(11 + call, si.stream_id("tokens", 500), rows * vocab, 1.0)
        logits = si.bf16_bits_to_f32(bits).reshape(rows, vocab).copy()          # bf16-valued: ties do occur
        if vocab > 2:
            logits[0, :] = 0.25                                                # a row of ties: lowest ids win
            logits[rows - 1, vocab - 1] = 9.0                                  # the winner sits in the ragged tail
        d_logits = torch.from_numpy(logits).cuda()
        ids.fill_(-1)
        firp_topb_static(d_logits.data_ptr(), rows, vocab, b, ids.data_ptr(), vals.data_ptr(), stream)
        torch.cuda.synchronize()
        got_ids, got_vals = ids.cpu().numpy(), vals.cpu().numpy()
        bb = min(b, vocab)
        check = sorted(set([0, rows - 1] + list(range(0, rows, max(1, rows // 64)))))
        for r in check:
            want = np.lexsort((np.arange(vocab), -logits[r]))[:bb]
            assert np.array_equal(got_ids[r, :bb], want), "row %d (call %d)" % (r, call)
            assert np.array_equal(got_vals[r, :bb], logits[r][want])
    # a vocabulary whose segment count does not fit 32 bits of intermediate arithmetic is refused, not wrapped
    with pytest.raises(FirpError) as e:
        firp_topb_static(d_logits.data_ptr(), 1, 2 ** 31 - 1, b, ids.data_ptr(), vals.data_ptr(), stream)
    assert e.value.code == binding.FIRP_ERR_CAPACITY
