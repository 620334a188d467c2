"""CPU-side checks of the C-ABI library: it builds, loads, and exports every symbol the header
declares.  No kernel runs here."""
import ctypes as C
import os
import re

from paper_2510_13797_b200 import binding as B
from paper_2510_13797_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "breadcrumbs.h")).read()
    return sorted(set(re.findall(r"^BC_API [\w \*]+?\b(bc_\w+)\(", text, flags=re.M)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build_library()
    assert os.path.exists(path)
    handle = C.CDLL(path)
    names = _declared()
    assert len(names) >= 20
    for name in names:
        assert hasattr(handle, name), f"{name} is declared in breadcrumbs.h but not exported"
    # the binding covers exactly the declared set
    assert sorted(B.SYMBOLS) == names


def test_version_status_strings_and_size_query():
    lib = B.lib()
    assert lib.bc_version() >= 100
    assert lib.bc_status_string(0) == b"BC_OK"
    assert lib.bc_status_string(B.BC_ERR_NO_PAGES) == b"BC_ERR_NO_PAGES"
    cfg = B.BcConfig(layers=2, kv_heads=8, q_heads=32, head_dim=128, c_default=16, page_size=16, max_seqs=64,
                     num_pages=1000, max_pages_per_seq=100, max_entries_per_seq=0, flags=0)
    sizes = [C.c_size_t() for _ in range(3)]
    assert lib.bc_cache_query_bytes(C.byref(cfg), *[C.byref(s) for s in sizes]) == B.BC_OK
    entry = 2 * 8 * 128 * 2
    assert sizes[0].value == 2 * 1000 * 16 * entry
    assert sizes[1].value >= 4 * (1000 + 64 * 100) and sizes[2].value > 0
    # invalid and unsupported configurations are refused on the host
    for field, value, want in (("page_size", 0, B.BC_ERR_INVALID_ARG), ("q_heads", 30, B.BC_ERR_INVALID_ARG),
                               ("head_dim", 96, B.BC_ERR_UNSUPPORTED), ("kv_heads", 16, B.BC_ERR_UNSUPPORTED)):
        bad = B.BcConfig.from_buffer_copy(cfg)
        setattr(bad, field, value)
        if field == "kv_heads":
            bad.q_heads = 16
        assert lib.bc_cache_query_bytes(C.byref(bad), *[C.byref(s) for s in sizes]) == want, field
    assert lib.bc_cache_query_bytes(None, *[C.byref(s) for s in sizes]) == B.BC_ERR_INVALID_ARG
    # null handles are refused, not dereferenced
    assert lib.bc_cache_destroy(None) == B.BC_ERR_INVALID_ARG
    assert lib.bc_kernel_launches(None) == 0
