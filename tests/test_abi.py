"""The C-ABI library loads and exports every symbol that include/ziplm.h declares (no GPU)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2302_04089_b200 import build
    return ctypes.CDLL(build.build())


def declared_symbols():
    src = open(os.path.join(ROOT, "include", "ziplm.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(ziplm_[a-z_0-9]+)\s*\(", src)))


def test_header_declares_the_expected_entry_points():
    syms = declared_symbols()
    for name in ("ziplm_hessian_accumulate", "ziplm_prune_layers", "ziplm_damped_inverse",
                 "ziplm_hessian_workspace_bytes", "ziplm_prune_workspace_bytes",
                 "ziplm_inverse_workspace_bytes", "ziplm_status_string",
                 "ziplm_hessian_accumulate_tokens", "ziplm_hessian_tokens_workspace_bytes",
                 "ziplm_kept_structures", "ziplm_gather_columns", "ziplm_gather_rows",
                 "ziplm_select_levels", "ziplm_select_workspace_bytes", "ziplm_search_levels",
                 "ziplm_search_workspace_bytes", "ziplm_damped_inverse_noalloc"):
        assert name in syms


def test_library_exports_every_declared_symbol(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), name


def test_status_strings_and_workspace_queries(lib):
    lib.ziplm_status_string.restype = ctypes.c_char_p
    names = [lib.ziplm_status_string(i).decode() for i in range(8)]
    assert names[0] == "ZIPLM_OK" and len(set(names)) == 8
    lib.ziplm_prune_workspace_bytes.restype = ctypes.c_size_t
    lib.ziplm_inverse_workspace_bytes.restype = ctypes.c_size_t
    a = lib.ziplm_prune_workspace_bytes(1, 64, 256, 1, 3)
    b = lib.ziplm_prune_workspace_bytes(12, 768, 3072, 1, 12)
    assert 0 < a < b and a % 256 == 0 and b % 256 == 0
    assert lib.ziplm_prune_workspace_bytes(1, 64, 255, 64, 3) == 0     # 255 % 64 != 0
    assert lib.ziplm_inverse_workspace_bytes(2, 100) >= 2 * 2 * 128 * 128 * 8
    lib.ziplm_select_workspace_bytes.restype = ctypes.c_size_t
    lib.ziplm_search_workspace_bytes.restype = ctypes.c_size_t
    assert lib.ziplm_select_workspace_bytes(3, 24, 10000) >= 3 * 24 * 10001
    assert lib.ziplm_search_workspace_bytes(3, 24, 10000) > lib.ziplm_select_workspace_bytes(3, 24, 10000)
    assert lib.ziplm_select_workspace_bytes(0, 24, 10000) == 0


def test_options_round_trip_and_reject_bad_values(lib):
    lib.ziplm_set_option.restype = ctypes.c_int
    lib.ziplm_get_option.restype = ctypes.c_int
    for opt, good, bad in ((0, 1, 2), (1, 8, 9), (2, 1, 2), (3, 1, 5), (4, 1000, -1), (5, 1, 2)):
        assert lib.ziplm_get_option(opt) == 0
        assert lib.ziplm_set_option(opt, good) == 0 and lib.ziplm_get_option(opt) == good
        assert lib.ziplm_set_option(opt, bad) == 1 and lib.ziplm_get_option(opt) == good
        assert lib.ziplm_set_option(opt, 0) == 0
    assert lib.ziplm_set_option(6, 0) == 1 and lib.ziplm_set_option(-1, 0) == 1
    assert lib.ziplm_get_option(17) == 0


def test_prune_layers_rejects_a_misaligned_hessian_on_the_host(lib):
    """H is read with 128-bit loads: a pointer that is not 16-byte aligned is refused before
    anything is enqueued (only the return code is looked at; nothing is launched)."""
    lib.ziplm_prune_layers.restype = ctypes.c_int
    lib.ziplm_prune_layers.argtypes = [ctypes.c_void_p] * 2 + [ctypes.c_int] * 4 + [ctypes.c_float] + \
        [ctypes.c_void_p, ctypes.c_int] + [ctypes.c_void_p] * 7 + [ctypes.c_size_t, ctypes.c_void_p]
    levels = (ctypes.c_int * 1)(4)
    base = 1 << 20                       # never dereferenced: the call stops at the argument checks

    def call(h_addr):
        return lib.ziplm_prune_layers(base, h_addr, 1, 8, 8, 1, 0.01, levels, 1, base, base, None,
                                      base, None, base, None, 0, None)

    assert call(base + 4096 + 4) == 1            # ZIPLM_ERR_INVALID_ARG
    assert call(base + 4096 + 8) == 1
    assert call(base + 4096) == 2                # aligned: next check is the (missing) workspace


def test_binding_mirrors_the_abi_names():
    import paper_2302_04089_b200 as z
    for name in declared_symbols():
        assert hasattr(z, name[len("ziplm_"):]), name


def test_compute_entry_points_fail_loudly_without_a_device(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    lib.ziplm_damped_inverse.restype = ctypes.c_int
    buf = (ctypes.c_char * 4096)()
    addr = (ctypes.addressof(buf) + 255) // 256 * 256
    # invalid arguments are still reported first
    assert lib.ziplm_damped_inverse(None, 1, 4, ctypes.c_float(0.01), None, None, None, 0, None) == 1
