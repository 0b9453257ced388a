"""CPU-only: the CUDA library builds, loads and exports every function include/memstore.h declares
(no compute call is made here), and the binding refuses to run without it."""
import ctypes
import re
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent


def declared_functions():
    text = (ROOT / "include" / "memstore.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(memstore_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2607_27090_b200 import build, memstore

    lib_path = build.build()
    names = declared_functions()
    assert len(names) >= 10 and "memstore_inject" in names and "memstore_retrieve" in names
    lib = ctypes.CDLL(str(lib_path))
    for n in names:
        assert hasattr(lib, n), f"{n} declared in memstore.h but not exported"
    assert set(memstore.EXPORTS) == set(names)
    assert memstore.load_library().memstore_version().decode().endswith("sm_100a")


def test_struct_layouts_match_header_sizes():
    # the ctypes mirrors must have the C sizes (x86-64 / LP64): config 112 bytes, cache 72, stats 80
    from paper_2607_27090_b200 import memstore

    assert ctypes.sizeof(memstore._Config) == 112
    assert ctypes.sizeof(memstore._PagedCache) == 72
    assert ctypes.sizeof(memstore._Stats) == 152


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    import pytest

    from paper_2607_27090_b200 import memstore

    monkeypatch.setattr(memstore, "_lib", None)
    monkeypatch.setattr(memstore, "_LIB_PATH", tmp_path / "libmemstore.so")
    with pytest.raises(ImportError):
        memstore.load_library()


def test_product_path_does_not_import_the_oracle():
    for f in (ROOT / "paper_2607_27090_b200").rglob("*"):
        if f.suffix in (".py", ".cu", ".cuh", ".h"):
            src = f.read_text()
            assert "import oracle" not in src and "from oracle" not in src and "memoracle" not in src, f


def test_llama3_frequency_table_of_the_library_equals_the_oracles():
    """Host arithmetic inside the library (no GPU needed): the rescaled table must agree bit for bit with the
    oracle's independent evaluation, because a one-ulp difference in a frequency is visible at large positions."""
    import numpy as np

    import oracle
    from paper_2607_27090_b200 import memstore

    for R, theta, args in ((128, 5e5, (8.0, 1.0, 4.0, 8192)), (64, 1e4, (4.0, 1.0, 4.0, 4096)), (96, 1e6, (32.0, 1.0, 4.0, 8192)),
                           (128, 5e5, (1.0, 1.0, 4.0, 8192))):  # fmt: skip
        got = np.array(memstore.rope_table_llama3(R, theta, *args), np.float32)
        want = oracle.inv_freq_llama3(R, theta, *args)
        assert np.array_equal(got, want)
    import pytest

    with pytest.raises(memstore.MemStoreError):
        memstore.rope_table_llama3(127, 5e5)


def test_header_is_plain_c_and_cpp_and_matches_the_struct_sizes(tmp_path):
    """include/memstore.h compiles as C99 and as C++11 with warnings as errors, and the C compiler's struct sizes are
    the ones the ctypes mirrors assume."""
    import subprocess

    src = tmp_path / "hdr.c"
    src.write_text(
        '#include "memstore.h"\n#include <stdio.h>\n'
        "int main(void) { printf(\"%zu %zu %zu %zu\\n\", sizeof(memstore_config), sizeof(ms_paged_cache), sizeof(memstore_stats_t),"
        " sizeof(ms_ann_params)); return 0; }\n"
    )
    inc = str(ROOT / "include")
    exe = tmp_path / "hdr"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-I", inc, str(src), "-o", str(exe)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()
    assert [int(x) for x in out] == [112, 72, 152, 16]
    subprocess.run(["g++", "-std=c++11", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only", "-x", "c++", "-I", inc, str(src)], check=True)
