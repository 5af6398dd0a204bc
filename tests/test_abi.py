"""The C-ABI library loads without a GPU and exports every symbol include/rpo.h declares."""
import ctypes
import os
import re

import paper_2601_19404_b200 as rpo
from paper_2601_19404_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "rpo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rpo_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_all_declared_symbols():
    build.build()
    lib = rpo.load_library()
    names = declared_symbols()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), f"{n} declared in rpo.h but not exported"
    assert sorted(binding.EXPORTED_SYMBOLS) == names


def test_host_only_calls_work_without_a_device():
    lib = rpo.load_library()
    assert lib.rpo_strerror(0) == b"ok" and b"KV" in lib.rpo_strerror(-3)
    s = rpo.shape_preset("qwen1.5b-class")
    assert (s.n_layers, s.d_model, s.n_q_heads, s.n_kv_heads, s.head_dim, s.d_ffn, s.vocab) == (28, 1536, 12, 2, 128, 8960, 151936)
    assert s.dtype == 1 and s.kv_block_tokens == 16
    t = rpo.shape_preset("tiny")
    assert (t.d_model, t.d_ffn, t.vocab, t.dtype) == (256, 688, 1024, 0)
    bad = binding.Shape()
    assert lib.rpo_shape_preset(b"nope", ctypes.byref(bad)) == -1
    assert lib.rpo_create(None, None, None, None) == -1


def test_presets_match_workload_table():
    import workloads
    for name, d in workloads.SHAPES.items():
        s = rpo.shape_preset(name)
        for k in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab"):
            assert getattr(s, k) == d[k]
        assert abs(s.rope_base - d["rope_base"]) < 1e-3 * d["rope_base"] and s.dtype == (1 if d["dtype"] == "bf16" else 0)


def test_no_device_fails_loudly():
    import torch
    if torch.cuda.is_available():
        return
    import pytest
    with pytest.raises(RuntimeError):
        rpo.Context(rpo.shape_preset("tiny"), 64, 4, 8, 256, 256)
    lib = rpo.load_library()
    h = ctypes.c_void_p()
    s = rpo.shape_preset("tiny"); lim = binding.Limits(64, 4, 8, 256, 256)
    assert lib.rpo_create(ctypes.byref(h), ctypes.byref(s), ctypes.byref(lim), None) == -4   # RPO_ERR_CUDA
