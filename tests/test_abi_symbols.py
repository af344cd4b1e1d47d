"""The C-ABI library builds, loads, and exports every symbol the header declares
(no compute calls: this runs without a GPU)."""
import ctypes
import os
import re

from paper_2508_18182_b200 import binding
from paper_2508_18182_b200.build import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "adloco.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(adloco_[a-z_]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    path = build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), f"{n} declared in adloco.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_binding_loads_and_reports_status_strings():
    lib = binding.load_library()
    assert lib.adloco_status_string(0) == b"ok"
    assert b"invalid" in lib.adloco_status_string(binding.ERR_INVALID_ARG)
    assert lib.adloco_launch_count(None) == 0


def test_check_merge_host_logic():
    # CheckMerge (Algorithm 1): the w trainers with the smallest requested batch
    assert binding.check_merge([8, 2, 5, 2], 2) == [1, 3]
    assert binding.check_merge([8, 2, 5, 2], 0) == []
    assert binding.check_merge([8], 1) == []
    assert binding.check_merge([8, 2], 3) == []
    assert binding.check_merge([8, 2, 5], 3) == [1, 2, 0]
    import oracle.adloco_oracle as O
    import random
    rnd = random.Random(3)
    for _ in range(200):
        k = rnd.randint(0, 9)
        b = [rnd.randint(1, 6) for _ in range(k)]
        w = rnd.randint(0, 10)
        assert binding.check_merge(b, w) == O.check_merge(b, w)
