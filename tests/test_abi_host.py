"""Host-side checks of the C-ABI library that need no GPU."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2308_15030_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "swapmoe.h")).read()
    declared = sorted(set(re.findall(r"\b(swapmoe_[a-z_]+)\s*\(", hdr)))
    assert len(declared) >= 14
    L = binding.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert sorted(binding.EXPORTS) == declared


def test_status_strings():
    assert binding.status_string(0) == "ok"
    for s in range(-7, 0):
        assert binding.status_string(s) not in ("ok", "unknown status")
    assert binding.status_string(-99) == "unknown status"


def test_topk_importance_host():
    assert binding.topk_importance([1, 5, 5, 0.5, 7, 5], 3).tolist() == [4, 1, 2]
    assert binding.topk_importance(np.zeros(5), 2).tolist() == [0, 1]
    with pytest.raises(binding.SwapMoEError):
        binding.topk_importance([1.0, 2.0], 3)


def test_create_rejects_bad_config_before_touching_the_device():
    L = binding.lib()
    h = ctypes.c_void_p()
    for kw in (dict(K=9), dict(top_k=2, K=1), dict(dtype=3), dict(act=2), dict(max_tokens=0)):
        base = dict(E=8, d_model=128, d_ff=256, top_k=1, K=4, dtype=1, act=0, renorm_topk=0,
                    max_tokens=16, spare_slots=0)
        base.update(kw)
        c = binding.Config(**base)
        assert L.swapmoe_create(ctypes.byref(h), ctypes.byref(c)) == -1
    assert L.swapmoe_create(None, None) == -1


def test_no_silent_cpu_fallback():
    """Without a GPU create() must fail loudly rather than compute on the host."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(binding.SwapMoEError) as e:
        binding.Layer(8, 128, 256, 1, 4, binding.BF16, max_tokens=16)
    assert e.value.status in (-5, -7)
