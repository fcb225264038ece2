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


def test_cost_model_reproduces_the_paper_tables():
    # the library's own cost model against the size / FLOP columns the paper prints (Table 1, Table 4
    # and the headline ratios), read from the golden file
    entry.build()
    import paper_2206_15014_b200 as nm
    rows = [ln.split() for ln in open(os.path.join(ROOT, "tests", "golden", "paper_tables.txt")) if ln.strip() and not ln.startswith("#")]
    cfg_of = {"Q4": (4, 4, 4), "Q8": (4, 4, 8), "S4": (2, 4, 4), "S8": (2, 4, 8)}
    seen = 0
    for r in rows:
        if r[0] != "table4":
            continue
        comp, red = nm.nm_encoder_cost([cfg_of[c] for c in r[2:8]], index_bits=2)
        assert round(100 * comp, 1) == float(r[8]), r
        if r[9] != "-":
            assert round(100 * red, 1) == float(r[9]), r
        seen += 1
    assert seen >= 8
    head = {r[1]: float(r[2]) for r in rows if r[0] == "headline"}
    assert 100 * (1 - nm.nm_bits_per_param(2, 4, 4, 0) / 32) == head["sparse_q4"]
    assert 100 * (1 - nm.nm_bits_per_param(4, 4, 4) / 32) == head["dense_q4"]
    # stored sizes agree with the model at this library's field widths
    for n, m, bits in [(2, 4, 8), (1, 4, 4), (2, 8, 8), (1, 8, 4), (4, 8, 8), (4, 4, 4)]:
        vb, mb = nm.nm_packed_sizes(768, 3072, n, m, bits)
        assert (vb + mb) * 8 == 768 * 3072 * nm.nm_bits_per_param(n, m, bits)
    assert nm.nm_bits_per_param(3, 2, 8) == -1.0
    # 1:4 and 2:8 run on the 2-of-4 path, 4:8 does not
    assert nm.nm_encoder_cost([(1, 4, 8)] * 6)[1] == 0.5 and nm.nm_encoder_cost([(4, 8, 8)] * 6)[1] == 0.0


def test_pair_tile_plan_covers_every_tile_once_in_balanced_ranges():
    entry.build()
    import pytest
    import paper_2206_15014_b200 as nm
    for n_tok, n_out, pairs, resident, req in [(86, 16, 74, True, 0), (86, 12, 74, True, 0), (86, 4, 74, False, 0),
                                               (86, 4, 74, False, 1), (86, 4, 74, False, 9), (10, 8, 74, False, 0),
                                               (7, 3, 21, True, 0), (1, 1, 1, False, 0), (33, 5, 64, False, 200)]:
        band, start, to, tt = nm.nm_pair_tile_plan(n_tok, n_out, pairs, resident, req)
        n = n_tok * n_out
        assert 1 <= band <= n_tok and (band == n_tok if resident else True)
        # the numbering is a bijection onto the grid, band by band, output-tile-major inside a band
        assert sorted(zip(to, tt)) == [(o, t) for o in range(n_out) for t in range(n_tok)]
        for t in range(1, n):
            same_band = tt[t] // band == tt[t - 1] // band
            assert (to[t], tt[t]) > (to[t - 1], tt[t - 1]) if same_band else tt[t] // band == tt[t - 1] // band + 1
        # contiguous, non-empty ranges that cover everything
        assert start[0] == 0 and start[-1] == n and all(b > a for a, b in zip(start, start[1:]))
        # equal cost up to one tile and one crossing
        crossing = 1.0 if resident else 0.2
        costs = [(b - a) + crossing * sum(1 for t in range(a + 1, b) if to[t] != to[t - 1]) for a, b in zip(start, start[1:])]
        assert max(costs) - min(costs) <= 1.0 + 2 * crossing + 1e-9, (n_tok, n_out, pairs, costs)
    for bad in [(0, 4, 2), (4, 4, 17), (4, 4, 200)]:
        start = (ctypes.c_int * 300)()
        lib = ctypes.CDLL(nm.LIB_PATH)
        assert lib.nm_pair_tile_plan(bad[0], bad[1], bad[2], 0, 0, start, None, None) < 0


def test_header_is_plain_c():
    # the boundary is a C ABI: the header must compile as C99 on its own, with warnings as errors
    import subprocess
    import tempfile
    with tempfile.TemporaryDirectory() as d:
        src = os.path.join(d, "t.c")
        open(src, "w").write('#include "nmsparse.h"\nint main(void) { return nm_version() > 0 ? 0 : 1; }\n')
        subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
                               "-c", src, "-o", os.path.join(d, "t.o")])
