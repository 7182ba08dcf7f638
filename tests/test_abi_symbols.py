"""The C-ABI library loads and exports every entry point include/bmu.h declares,
and its host-side argument checks answer without touching a GPU."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_05138_b200 import build, binding
    build.build_library()
    return binding.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "bmu.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"BMU_API\s+[\w\s\*]+?\b(bmu_\w+)\s*\(", text)))


def test_header_and_binding_agree(lib):
    from paper_2609_05138_b200 import binding
    names = declared_functions()
    assert len(names) >= 10
    assert sorted(binding.EXPORTS) == names
    for n in names:
        assert getattr(lib, n) is not None           # dlsym succeeds


def test_only_the_api_is_exported():
    import subprocess
    from paper_2609_05138_b200 import binding
    out = subprocess.check_output(["nm", "-D", "--defined-only", binding.LIB_PATH], text=True)
    syms = [l.split()[-1] for l in out.splitlines() if " T " in l]
    assert sorted(syms) == declared_functions()


def test_status_strings_and_version(lib):
    assert lib.bmu_status_string(0) == b"ok"
    assert b"workspace" in lib.bmu_status_string(3)
    assert lib.bmu_version() >= 100


def test_workspace_size_is_monotone(lib):
    f = lib.bmu_search_workspace_bytes
    a = f(4096, 1024, 10_000, 640_000, None)
    b = f(16384, 262144, 2_000_000, 160_000_000, None)
    assert 0 < a < b
    assert a % 256 == 0 and b >= 262144 * 4 + 2_000_000 * 8


def test_argument_checks_need_no_gpu(lib):
    # sizes are checked before any CUDA call is made
    assert lib.bmu_codebook_norms(None, -1, 4, None, None) == 1
    assert lib.bmu_search(None, 4, 1 << 30, None, None, 1, None, None, None) == 2
    assert b"limits" in lib.bmu_last_error()
    assert lib.bmu_search_ws(None, 4, 4, None, None, None, 0, 0, None, None, None, None, 0,
                             None) == 0           # N == 0: nothing to do
    assert lib.bmu_search_ws(None, 4, 4, None, None, None, 3, 0, None, None, None, None, 0,
                             None) == 1           # null pointers
    from paper_2609_05138_b200 import Opts
    o = Opts()
    o.vec = 3
    assert lib.bmu_search_ws(None, 4, 4, None, None, None, 3, 0, None, None,
                             ctypes.byref(o), None, 0, None) == 1


def test_describe_search_needs_no_gpu_and_names_the_kernel(lib):
    """bmu_describe_search is host logic: the benchmark shapes route as documented (large
    sweeps take the tensor-core sweep, the small one the planned kernel) and the launch count
    follows from the chunk."""
    from paper_2609_05138_b200 import Opts, SearchDesc
    d = SearchDesc()
    shapes = {"cfg1": (4096, 1024, 10_000, 640_000), "cfg2": (16384, 4096, 1_000_000, 80_000_000),
              "cfg4": (16384, 262144, 2_000_000, 160_000_000)}
    for name, (D, M, N, nnz) in shapes.items():
        assert lib.bmu_describe_search(D, M, N, nnz, None, ctypes.byref(d)) == 0
        assert d.kernel == (3 if name == "cfg1" else 6)
        assert d.head_rows == (0 if name == "cfg1" else 640)
        assert d.docs_per_block == (16 if name == "cfg1" else 128)
        assert d.chunk_neurons % d.slab == 0 and d.ragged_neurons == 0
        assert d.sweep_launches == -(-M // d.chunk_neurons)
    o = Opts()
    o.kernel, o.chunk_neurons = 6, 2048
    assert lib.bmu_describe_search(16384, 262144 + 36, 1000, 80_000, ctypes.byref(o), ctypes.byref(d)) == 0
    assert (d.kernel, d.chunk_neurons, d.sweep_launches, d.ragged_neurons, d.repack) == (6, 2048, 128, 36, 1)
    o.kernel = 6
    assert lib.bmu_describe_search(32, 1024, 10, 100, ctypes.byref(o), ctypes.byref(d)) == 2   # D < head
    assert lib.bmu_describe_search(32, 1024, 10, 100, None, None) == 1


def test_status_words_map_to_errors_without_a_gpu(lib):
    """The host entry points that read a search's status word back (bmu_search_host,
    bmu_search_batches_host, bmu_plan_create, bmu_last_status) turn it into an error through
    this mapping: a clean word is no error, a failed size check of the tiling pass is a
    workspace error, a wait that ran out a timeout."""
    assert lib.bmu_status_of_word(0) == 0
    assert lib.bmu_status_of_word(64) == 3 and b"tiling pass" in lib.bmu_last_error()
    assert lib.bmu_status_of_word(64 | 8) == 3
    for word in (1, 2, 4, 8, 16, 32):
        assert lib.bmu_status_of_word(word) == 5
        assert b"wait ran out" in lib.bmu_last_error() and str(word).encode() in lib.bmu_last_error()
    assert lib.bmu_status_of_word(128) == 5
