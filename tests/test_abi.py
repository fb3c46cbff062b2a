"""The C-ABI library loads without a GPU, exports every function the header
declares, and rejects bad parameters on the host before any CUDA call."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "fedhe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(he_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    import paper_2303_10837_b200 as he
    lib = ctypes.CDLL(he.LIB_PATH)
    names = declared_functions()
    assert len(names) >= 25
    for name in names:
        assert hasattr(lib, name), name
        assert name in he.EXPORTS, name + " has no binding"
    for name in he.EXPORTS:
        assert name in names, name + " is bound but not declared"


def test_error_strings_and_host_side_parameter_checks():
    import paper_2303_10837_b200 as he
    import synthetic_inputs as si
    assert he.he_strerror(0) == "ok"
    assert "parameter" in he.he_strerror(he.HE_ERR_PARAMS)
    bad = [
        (8192, [5, 7], 40),                                   # tiny moduli
        (8192, [si.PRIMES_N8192[0] + 2, si.PRIMES_N8192[1]], 40),   # not prime
        (8190, list(si.PRIMES_N8192), 40),                    # N not a power of two
        (32768, list(si.PRIMES_N8192), 40),                   # q != 1 mod 2N
        (8192, [si.PRIMES_N8192[0], si.PRIMES_N8192[0]], 40), # repeated
        (8192, list(si.PRIMES_N8192), 59),                    # scale >= q0 / 4
        (8192, [si.PRIMES_N8192[0]], 40),                     # a single prime leaves nothing after the rescale
        (4096, list(si.PRIMES_N8192), 40),                    # N below the supported range
        (8192, [0x3fffffffffff0001, si.PRIMES_N8192[1]], 40),  # a prime (= 1 mod 2N) of 62 bits: lazy values must stay below 2^63
    ]
    for N, primes, ld in bad:
        with pytest.raises(he.HeError) as ei:
            he.he_ctx_create(N, primes, ld)
        assert ei.value.code == he.HE_ERR_PARAMS


def test_missing_library_is_a_loud_error(tmp_path, monkeypatch):
    import importlib.util
    import paper_2303_10837_b200 as he
    src = os.path.join(os.path.dirname(he.__file__), "__init__.py")
    pkg = tmp_path / "he_copy"
    pkg.mkdir()
    (pkg / "__init__.py").write_text(open(src).read())
    spec = importlib.util.spec_from_file_location("he_copy", str(pkg / "__init__.py"))
    mod = importlib.util.module_from_spec(spec)
    with pytest.raises(ImportError):
        spec.loader.exec_module(mod)
