"""The C-ABI library loads and exports every symbol include/gram.h declares (no GPU needed)."""
import ctypes
import os
import re

from paper_2204_04179_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "gram.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gram_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    import __graft_entry__
    __graft_entry__.build()
    L = ctypes.CDLL(binding.LIB_PATH)
    names = declared_symbols()
    assert len(names) >= 20
    for n in names:
        assert hasattr(L, n), n
    assert sorted(binding.SYMBOLS) == names


def test_config_struct_matches_header_field_order():
    text = open(os.path.join(ROOT, "include", "gram.h")).read()
    body = re.search(r"typedef struct gram_config \{(.*?)\} gram_config;", text, re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = []
    for decl in body.split(";"):
        decl = decl.strip()
        if not decl:
            continue
        typ, rest = decl.split(None, 1)
        fields += [(f.strip(), typ) for f in rest.split(",")]
    ctype = {"int32_t": ctypes.c_int32, "int64_t": ctypes.c_int64, "float": ctypes.c_float}
    assert [(n, ctype[t]) for n, t in fields] == list(binding.GramConfig._fields_)
    body = re.search(r"typedef struct gram_step_report \{(.*?)\} gram_step_report;", text, re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = []
    for decl in body.split(";"):
        decl = decl.strip()
        if decl:
            typ, rest = decl.split(None, 1)
            fields += [(f.strip(), typ) for f in rest.split(",")]
    assert [(n, ctype[t]) for n, t in fields] == list(binding.GramStepReport._fields_)


def test_noam_rate_host_function_matches_the_oracle():
    """Host logic, no GPU: the library's learning-rate curve against the oracle's (fp32 result of a double formula)."""
    from oracle import gram_oracle as O
    for warm in (0, 1, 7, 4000):
        for t in (1, 2, 6, 7, 8, 100, 3999, 4000, 4001, 10**6):
            got = binding.noam_rate(t, 1e-4, warm)
            assert abs(got - O.noam_rate(t, 1e-4, warm)) <= 1e-7 * 1e-4 + 6e-8 * got
