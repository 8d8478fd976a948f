"""No-GPU checks: the C-ABI library loads, exports every symbol the header declares, and the host-side
network helpers behave."""
import ctypes
import os
import re

import pytest

from paper_1804_10574_b200 import nets

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ddg.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ddg_[a-z0-9_]+)\s*\(", text)))


def test_library_loads_and_exports_every_declared_symbol():
    from paper_1804_10574_b200 import build
    build.build()
    from paper_1804_10574_b200 import binding
    names = declared_symbols()
    assert len(names) >= 20
    for n in names:
        assert hasattr(binding.lib(), n), n
    assert sorted(binding.EXPORTS) == names


def test_create_fails_loudly_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_1804_10574_b200 import binding
    with pytest.raises(binding.DdgError) as e:
        binding.Ddg(nets.mlp(), [1], 4, (64, 1, 1), 10)
    assert e.value.status == 5 and "no CUDA device" in str(e.value)


def test_product_path_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_1804_10574_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                assert "oracle" not in open(os.path.join(dirpath, f)).read().lower().replace("oracle's", ""), f


def test_split_helper():
    L = nets.resnet(18, 100)
    assert nets.split_even_blocks(L, 1) == []
    s = nets.split_even_blocks(L, 4)
    blocks = [i for i, l in enumerate(L) if l[0] == nets.BASIC_BLOCK]
    bounds = [-1] + s + [len(L) - 1]
    counts = [sum(1 for b in blocks if bounds[k] < b <= bounds[k + 1]) for k in range(4)]
    assert counts == [14, 14, 13, 13]
    with pytest.raises(ValueError):
        nets.split_even_blocks(nets.resnet(1, 10), 4)
    assert nets.config("resnet8")["split_after"] == [2]      # {stem, block 1} | {block 2, block 3, pool, FC}
