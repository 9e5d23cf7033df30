"""CPU-side checks of the boundary: the C-ABI library builds, loads without a GPU and
exports every symbol include/mtmc_fused.h declares; the Python binding lists the same
names.  No compute call is made here."""
import ctypes
import os
import re

from paper_2511_20100_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "mtmc_fused.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mtmc_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_three_named_calls():
    names = declared_symbols()
    for n in ("mtmc_fused_linear", "mtmc_swiglu", "mtmc_linear_lse"):
        assert n in names


def test_library_builds_loads_and_exports_every_declared_symbol():
    path = build.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    for name in declared_symbols():
        assert hasattr(lib, name), "missing export: %s" % name
    lib.mtmc_version.restype = ctypes.c_int
    assert lib.mtmc_version() >= 100


def test_debug_build_variants_compile_and_say_what_they_are():
    """The trace build (-DMTMC_TRACE) and the index-check build (-DMTMC_CHECKS) compile for sm_100a and export the same
    symbols; only the trace build reports tracing as available."""
    plain = ctypes.CDLL(build.build())
    plain.mtmc_trace_enabled.restype = ctypes.c_int
    assert plain.mtmc_trace_enabled() == 0
    for variant in ("trace", "checks"):
        lib = ctypes.CDLL(build.build(variant=variant))
        for name in declared_symbols():
            assert hasattr(lib, name), "%s build: missing export %s" % (variant, name)
        lib.mtmc_trace_enabled.restype = ctypes.c_int
        assert lib.mtmc_trace_enabled() == (1 if variant == "trace" else 0)


def test_binding_covers_the_header():
    assert sorted(binding.EXPORTS) == declared_symbols()
    for name in binding.EXPORTS:
        if name not in ("mtmc_set_stream", "mtmc_last_error"):
            assert hasattr(binding, name), name


def test_product_path_has_no_oracle_or_cpu_fallback():
    pkg = os.path.join(ROOT, "paper_2511_20100_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle\b", src, flags=re.M), "%s imports the oracle" % f
                assert "mtmc_ref" not in src and "libmtmcref" not in src, "%s reaches for the oracle library" % f
