"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import __graft_entry__ as entry

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "nmsparse.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(nm_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    entry.build()
    import paper_2206_15014_b200 as nm
    lib = ctypes.CDLL(nm.LIB_PATH)
    names = _declared()
    assert len(names) >= 15
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in nmsparse.h but not exported"
    assert set(names) == set(nm.EXPORTS)


def test_host_only_entry_points():
    entry.build()
    import paper_2206_15014_b200 as nm
    assert nm.nm_version() >= 100
    assert nm.nm_packed_sizes(768, 768, 2, 4, 8) == (768 * 384, 768 * 24 * 4)
    assert nm.nm_packed_sizes(768, 768, 2, 4, 4) == (768 * 192, 768 * 24 * 4)
    assert nm.nm_packed_sizes(4, 8, 1, 4, 4) == (4, 4 * 4)       # 4 meta bits per row, padded to a word
    assert nm.nm_packed_sizes(4, 16, 4, 8, 8) == (32, 4 * 4)
    assert nm.nm_packed_sizes(4, 16, 4, 4, 8) == (64, 0)
    assert nm.nm_pack_workspace_bytes(0) == 0 and nm.nm_pack_workspace_bytes(96) > 0
    assert "NULL" in nm.nm_strerror(nm.NM_ERR_NULL)
    for code in range(-8, 1):
        assert nm.nm_strerror(code) != "unknown nmsparse code"
    assert nm.nm_int_linear_check(4096, 768, 768, 2, 4, 8) == nm.NM_OK
