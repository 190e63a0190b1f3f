"""The C-ABI library loads and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "kvzap.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kvzap_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2601_07891_b200 import binding
    lib = binding.load()
    declared = _declared_symbols()
    assert len(declared) >= 9
    for name in declared:
        assert hasattr(lib, name), "libkvzap.so does not export %s" % name
    # the binding covers the same set
    assert sorted(binding.SIGNATURES) == declared


def test_create_rejects_bad_shapes_before_touching_the_device():
    from paper_2601_07891_b200 import binding
    lib = binding.load()
    for kwargs, needle in [
        (dict(d_model=100), "d_model"),
        (dict(hidden=96), "hidden"),
        (dict(hidden=640 + 64), "hidden"),
        (dict(n_kv_heads=9), "n_kv_heads"),
        (dict(head_dim=12), "head_dim"),
        (dict(max_tokens=0), "max_tokens"),
    ]:
        base = dict(d_model=4096, hidden=512, n_kv_heads=8, head_dim=128, n_layers=1, max_tokens=4096, max_seqs=1)
        base.update(kwargs)
        with pytest.raises(binding.KvzapError) as ei:
            binding.kvzap_create(**base)
        assert ei.value.status in (1, 2) and needle in str(ei.value)
    assert lib.kvzap_destroy(None) == 0
    assert lib.kvzap_launch_count(None) == 0


def test_no_cpu_fallback_create_fails_loudly_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2601_07891_b200 import binding
    with pytest.raises(binding.KvzapError) as ei:
        binding.kvzap_create(4096, 0, 8, 128, 1, 4096)
    assert ei.value.status == 3


def test_product_path_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2601_07891_b200")
    for dirpath, _dirs, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"(import\s+oracle|from\s+oracle|kvzap_oracle|oracle/)", src), f
