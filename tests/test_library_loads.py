"""The C-ABI library builds for sm_100a, loads without a GPU and exports what include/ada.h declares."""
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_every_declared_symbol_is_exported():
    import paper_2412_18910_b200 as pkg
    L = pkg.lib()
    header = open(os.path.join(ROOT, "include", "ada.h")).read()
    declared = set(re.findall(r"\b(ada_[a-z_0-9]+)\s*\(", header))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(L, name), name
    assert declared == set(pkg.exported_symbols)


def test_workspace_size_is_reported_without_a_gpu():
    import ctypes as C
    import paper_2412_18910_b200 as pkg
    L = pkg.lib()
    ok = pkg.Config(32, 4096, 32, 128, 11008, 32000, 1e4, 1e-6, 512, 10, 0, 1, 4096, 64)
    n = L.ada_workspace_bytes(C.byref(ok))
    assert 2 * 2 * 32 * 4096 * 4096 < n < 8 * 2**30          # at least the KV pool, well under 8 GiB
    bad = pkg.Config(32, 4096, 32, 128, 11008, 32000, 1e4, 1e-6, 512, 16, 0, 1, 4096, 64)   # n_max too large
    assert L.ada_workspace_bytes(C.byref(bad)) == 0


def test_scalar_predictor_configuration_is_validated():
    import ctypes as C
    import paper_2412_18910_b200 as pkg
    L = pkg.lib()
    base = (32, 4096, 32, 128, 11008, 32000, 1e4, 1e-6, 512, 10)
    assert L.ada_workspace_bytes(C.byref(pkg.Config(*base, 1, 1, 4096, 64, 2, 1))) > 0      # Eq. 3, k_min = 1
    assert L.ada_workspace_bytes(C.byref(pkg.Config(*base, 1, 1, 4096, 64, 2, 0))) == 0     # k_min below 1
    assert L.ada_workspace_bytes(C.byref(pkg.Config(*base, 1, 1, 4096, 64, 2, 11))) == 0    # k_min above n_max
    assert L.ada_workspace_bytes(C.byref(pkg.Config(*base, 1, 1, 4096, 64, 9, 1))) == 0     # too many blocks
    assert L.ada_workspace_bytes(C.byref(pkg.Config(*base, 2, 1, 4096, 64, 2, 1))) == 0     # unknown mode


def test_configurations_need_matrices_of_at_least_one_weight_box():
    """Prompts (every engine) and batches go through the multi-row tensor-core GEMM, whose weight boxes are 128 rows
    high: a model with a narrower matrix is refused at any batch size; the workspace of a batch-1 engine holds the
    128-row scratch of its prompt pass."""
    import ctypes as C
    import paper_2412_18910_b200 as pkg
    L = pkg.lib()
    narrow = (2, 64, 1, 64, 176, 4096, 1e4, 1e-6, 128, 8, 0)
    assert L.ada_workspace_bytes(C.byref(pkg.Config(*narrow, 1, 256, 64))) == 0
    assert L.ada_workspace_bytes(C.byref(pkg.Config(*narrow, 3, 256, 64))) == 0
    tiny = (2, 256, 4, 64, 688, 4096, 1e4, 1e-6, 128, 8, 0)
    one = L.ada_workspace_bytes(C.byref(pkg.Config(*tiny, 1, 256, 64)))
    three = L.ada_workspace_bytes(C.byref(pkg.Config(*tiny, 3, 256, 64)))
    assert one > 128 * (3 * 256) * 4 and three > one
