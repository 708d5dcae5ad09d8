"""The C ABI as a file: the shared library loads without a GPU and exports exactly the entry
points that include/aq_b200.h declares, and the Python binding covers the same set with the
same number of arguments.  No compute call is made here."""
import ctypes
import os
import re

import paper_2206_01299_b200 as aq
from paper_2206_01299_b200 import build as cuda_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "aq_b200.h")


def declared_functions():
    """name -> number of parameters, from the header (comments stripped)."""
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", " ", text, flags=re.S)
    text = text[text.index('extern "C"'):]
    out = {}
    for m in re.finditer(r"\b(aq_[a-z_0-9]+)\s*\(([^;{]*?)\)\s*;", text, flags=re.S):
        args = m.group(2).strip()
        out[m.group(1)] = 0 if args in ("", "void") else args.count(",") + 1
    return out


def test_header_declares_the_documented_entry_points():
    names = set(declared_functions())
    for required in ("aq_create", "aq_destroy", "aq_configure", "aq_encode", "aq_decode", "aq_quant_grad",
                     "aq_dequant_grad", "aq_state_checksum", "aq_status", "aq_last_error",
                     "aq_encode_host", "aq_decode_host", "aq_export_sample", "aq_import_sample",
                     "aq_state_checksum_noalloc"):
        assert required in names


def test_library_builds_loads_and_exports_every_declared_symbol():
    path = cuda_build.build()                      # compiles for sm_100a if the .so is stale; needs no GPU
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} is declared in the header but not exported"


def test_binding_matches_the_header():
    decl = declared_functions()
    assert set(aq.SIGNATURES) == set(decl)
    for name, (_, argtypes) in aq.SIGNATURES.items():
        assert len(argtypes) == decl[name], name
        assert callable(getattr(aq, name)), f"binding has no function {name}"


def test_constants_match_the_header():
    text = open(HEADER).read()
    for name in ("AQ_OK", "AQ_EINVAL", "AQ_ENOMEM", "AQ_ECUDA", "AQ_EUNSUPPORTED", "AQ_DTYPE", "AQ_BATCH",
                 "AQ_STREAM", "AQ_RAW", "AQ_FIRST_FLAGS", "AQ_ROWS_PER_CTA", "AQ_ROUNDING", "AQ_SEED", "AQ_EPOCH", "AQ_L2_PREFETCH",
                 "AQ_ROUND_INTERVAL", "AQ_ROUND_STOCHASTIC", "AQ_FP16", "AQ_BF16",
                 "AQ_ST_BAD_ID", "AQ_ST_DUP_ID", "AQ_ST_NO_RAW", "AQ_ST_STAGED", "AQ_ST_BAD_PTR", "AQ_RAW_LIST"):
        m = re.search(rf"\b{name}\s*=\s*(-?\d+)", text)
        assert m, name
        assert getattr(aq, name) == int(m.group(1)), name


def test_missing_library_is_an_error_not_a_fallback(monkeypatch):
    from paper_2206_01299_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", os.path.join(ROOT, "no_such_dir", "libaq_b200.so"))
    try:
        binding.lib()
    except RuntimeError as e:
        assert "no fallback" in str(e)
    else:
        raise AssertionError("a missing library must raise")
