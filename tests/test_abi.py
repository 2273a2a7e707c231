"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header declares,
and its host-side validation rejects bad calls before anything is launched."""
import ctypes
import os
import re

import pytest

import paper_2410_20488_b200 as firp
from paper_2410_20488_b200 import binding, build as firp_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    firp_build.build()
    return firp.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "firp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(firp_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = declared_symbols()
    assert len(names) >= 13
    for name in names:
        assert hasattr(lib, name), name
    assert set(names) == set(binding.EXPORTS)


def good_cfg(**kw):
    base = dict(n_layers=2, d_model=256, n_heads=4, n_kv_heads=4, head_dim=64, d_ffn=688, vocab=1024, rms_eps=1e-5,
                rope_theta=1e4, max_batch=1, max_ctx=256, max_tree=8, max_k=3, max_depth=3, top_b=8)
    base.update(kw)
    return firp.ModelCfg(**base)


def test_create_validates_configuration(lib):
    ctx = firp.firp_create(good_cfg())
    assert firp.firp_workspace_bytes(ctx) > 0
    assert firp.firp_kv_bytes(ctx) == 1 * 2 * 2 * 256 * 4 * 64 * 2
    firp.firp_destroy(ctx)
    for bad in (dict(head_dim=96), dict(n_heads=3, n_kv_heads=2), dict(max_tree=129), dict(max_k=9), dict(top_b=0),
                dict(top_b=9), dict(max_batch=0), dict(max_batch=4, max_tree=64), dict(d_model=192),
                dict(max_depth=16), dict(max_ctx=4)):
        with pytest.raises(firp.FirpError):
            firp.firp_create(good_cfg(**bad))


def test_calls_out_of_order_are_state_errors(lib):
    ctx = firp.firp_create(good_cfg())
    with pytest.raises(firp.FirpError) as e:
        firp.firp_step(ctx, 1, None, 1, [-1], 1, 0, 0, None)
    assert e.value.code == binding.FIRP_ERR_STATE and "bind" in str(e.value)
    with pytest.raises(firp.FirpError) as e:
        firp.firp_kv_commit(ctx, 1)
    assert e.value.code == binding.FIRP_ERR_STATE
    with pytest.raises(firp.FirpError) as e:
        firp.firp_bind_buffers(ctx, 0, 0)
    assert e.value.code == binding.FIRP_ERR_BAD_ARG
    with pytest.raises(firp.FirpError) as e:
        firp.firp_bind_buffers(ctx, 4096 + 8, 4096)        # misaligned workspace
    assert e.value.code == binding.FIRP_ERR_BAD_ARG
    firp.firp_destroy(ctx)


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", os.path.join(ROOT, "does_not_exist.so"))
    with pytest.raises(ImportError):
        binding.load_library()
