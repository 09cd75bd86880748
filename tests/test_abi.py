"""The C-ABI library builds, loads and exports every symbol include/ps.h declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ps.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ps_[a-z_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2002_00655_b200.build import build
    lib = ctypes.CDLL(build())
    names = declared_symbols()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in ps.h but not exported"


def test_binding_covers_every_declared_symbol_with_the_same_name():
    import paper_2002_00655_b200 as ps
    for n in declared_symbols():
        assert n in ps.binding.SIGNATURES, n
        assert callable(getattr(ps, n)), n


def test_host_side_checks_need_no_gpu():
    import paper_2002_00655_b200 as ps
    sz = ps.ps_query_sizes(ps.ps_config_t(1000, 8, 4, 300, 0), 4096)
    assert sz.store_bytes == 4 * 300 * 8 * 4 and sz.table_bytes == 8000
    assert sz.freelist_bytes >= 4 * 8 + 4 * 300 * 4 and sz.workspace_bytes > 4096 * (8 * 4 + 16)
    for bad in (ps.ps_config_t(0, 8, 1, 10, 0), ps.ps_config_t(10, 8, 2, 4, 0)):      # no keys; too few slots
        try:
            ps.ps_query_sizes(bad, 16)
            raise AssertionError("accepted a bad configuration")
        except ps.PSError as e:
            assert e.code == ps.PS_ERR_INVALID_ARG
    try:
        ps.ps_query_sizes(ps.ps_config_t(10, 6, 1, 10, 0), 16)                         # row_len not a multiple of 4
        raise AssertionError("accepted row_len 6")
    except ps.PSError as e:
        assert e.code == ps.PS_ERR_UNSUPPORTED
    assert ps.ps_status_string(ps.PS_ERR_CAPACITY) == "partition full"
