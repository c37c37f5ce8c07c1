"""The C-ABI library loads and exports every symbol the header declares
(no compute calls: runs without a GPU)."""
import ctypes
import os
import re

import __graft_entry__ as entry
from paper_2607_16339_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "lacache.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lacache_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_header_symbols():
    entry.build()
    lib = ctypes.CDLL(binding.LIB_PATH)
    names = _declared()
    assert len(names) >= 16
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == [n for n in names if n in binding.EXPORTS]
    assert set(names) - set(binding.EXPORTS) == set(), set(names) - set(binding.EXPORTS)
    lib.lacache_version.restype = ctypes.c_int
    assert lib.lacache_version() >= 100


def test_create_rejects_bad_configs_without_gpu():
    lib = binding.load()
    h = ctypes.c_void_p()
    pl = (ctypes.c_int32 * 1)(8)

    def cfg(**kw):
        base = dict(dtype=0, engine=0, n_q_heads=4, n_kv_heads=2, head_dim=128, rope_theta=1e4,
                    softmax_scale=0.0, batch=1, prompt_lens=pl, gen_len=32, block_len=16,
                    sc_tiles_per_chunk=0, out_dtype=binding.OUT_FP32, precision_mode=binding.PRECISION_SPLIT,
                    cache_granularity=binding.GRANULARITY_TOKEN)
        base.update(kw)
        return binding.LacacheConfig(*[base[f[0]] for f in binding.LacacheConfig._fields_])

    cases = [
        (cfg(head_dim=96), binding.ERR_UNSUPPORTED),
        (cfg(n_kv_heads=3), binding.ERR_SHAPE),
        (cfg(block_len=24), binding.ERR_SHAPE),
        (cfg(dtype=7), binding.ERR_UNSUPPORTED),
        (cfg(batch=0), binding.ERR_INVALID_ARG),
        (cfg(rope_theta=0.0), binding.ERR_INVALID_ARG),
        (cfg(engine=2, dtype=1), binding.ERR_UNSUPPORTED),
        (cfg(out_dtype=2), binding.ERR_INVALID_ARG),
        (cfg(precision_mode=2), binding.ERR_UNSUPPORTED),       # a split of the probabilities is not offered
        (cfg(precision_mode=4), binding.ERR_UNSUPPORTED),       # no such mode
        (cfg(cache_granularity=5), binding.ERR_INVALID_ARG),
        (cfg(cache_granularity=binding.GRANULARITY_TILE, dtype=1), binding.ERR_UNSUPPORTED),   # tcgen05 engine only
    ]
    for c, want in cases:
        st = lib.lacache_create(ctypes.byref(c), ctypes.byref(h))
        assert st == want, (st, want, lib.lacache_last_error(None))
        assert not h.value
        assert lib.lacache_last_error(None)
    assert lib.lacache_create(None, ctypes.byref(h)) == binding.ERR_INVALID_ARG
    assert lib.lacache_build(None, 0, None, None, None, None) == binding.ERR_INVALID_ARG


def test_producer_create_rejects_bad_configs_without_gpu():
    lib = binding.load()
    h = ctypes.c_void_p()
    dummy = 0x1000   # never dereferenced: validation fails first

    def cfg(**kw):
        base = dict(vocab=10, d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=128, rms_eps=1e-5,
                    max_tokens=32, embed=dummy, norm_weight=dummy, w_qkv=dummy)
        base.update(kw)
        return binding.LacacheQkvConfig(*[base[f[0]] for f in binding.LacacheQkvConfig._fields_])

    cases = [
        (cfg(head_dim=64), binding.ERR_UNSUPPORTED),
        (cfg(d_model=200), binding.ERR_SHAPE),
        (cfg(d_model=16384), binding.ERR_SHAPE),
        (cfg(n_kv_heads=3), binding.ERR_SHAPE),
        (cfg(max_tokens=0), binding.ERR_INVALID_ARG),
        (cfg(w_qkv=None), binding.ERR_INVALID_ARG),
        (cfg(embed=None), binding.ERR_INVALID_ARG),
        (cfg(norm_weight=0x1004), binding.ERR_INVALID_ARG),
    ]
    for c, want in cases:
        st = lib.lacache_qkv_create(ctypes.byref(c), ctypes.byref(h))
        assert st == want, (st, want, lib.lacache_qkv_last_error(None))
        assert not h.value and lib.lacache_qkv_last_error(None)
    assert lib.lacache_qkv_create(None, ctypes.byref(h)) == binding.ERR_INVALID_ARG
    assert lib.lacache_qkv_project(None, None, None, 0, None, None, None, None, None) == binding.ERR_INVALID_ARG
    assert lib.lacache_step_tokens(None, None, None, None, None, None, None) == binding.ERR_INVALID_ARG


def test_product_path_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2607_16339_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cuh")):
                src = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in src and "from oracle" not in src, f
                assert "lacache_oracle" not in src, f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            src = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2607_16339_b200" not in src and "liblacache.so" not in src, f
