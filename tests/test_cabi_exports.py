"""The C-ABI library loads without a GPU and exports every symbol adapt.h declares. CPU only."""
import ctypes
import os
import re

from paper_2107_13490_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "adapt.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(adapt_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_loads_and_exports_all_declared_symbols():
    path = build.build()
    lib = ctypes.CDLL(path)
    names = declared_symbols()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names
    for n in names:   # the Python binding carries the same names
        assert hasattr(binding, n) or n in ("adapt_status_string", "adapt_last_error")


def test_status_strings_and_version_need_no_gpu():
    L = binding.lib()
    assert binding.adapt_version().startswith("adapt-b200")
    texts = {L.adapt_status_string(i).decode() for i in range(6)}
    assert len(texts) == 6 and "ok" in texts
    assert L.adapt_status_string(99).decode() == "unknown status"
