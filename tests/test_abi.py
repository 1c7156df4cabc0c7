"""The C-ABI library builds, loads without a GPU and exports every symbol
that include/dkv.h declares.  No compute call is made here."""
import ctypes
import os
import re

from paper_2505_15781_b200 import binding as B
from paper_2505_15781_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "dkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dkv_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    build.build()
    lib = B.load()
    names = declared_functions()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), f"{n} declared in dkv.h but not exported"
    assert sorted(B.EXPORTS) == names


def test_host_only_calls():
    lib = B.load()
    assert lib.dkv_strerror(0) == b"ok"
    assert b"arena" in lib.dkv_strerror(-4)
    assert lib.dkv_gemm_workspace_bytes(10, 128) >= 2048 * 128 * 4
    assert lib.dkv_gemm_workspace_bytes(0, 128) == 0
    assert lib.dkv_cache_bytes(None, 1, 16, None) == 0
    assert lib.dkv_refresh(None, 0) == -1
    assert lib.dkv_model_create(None, None, None, 0, None, None) == -1
    assert lib.dkv_model_bytes(None) == 0


def test_a_handle_that_is_not_live_is_a_state_error():
    """A pointer that no create call returned (or that was destroyed) is refused before anything is
    read through it: DKV_E_STATE from every entry point that takes a handle."""
    lib = B.load()
    buf = ctypes.create_string_buffer(4096)
    bogus = ctypes.c_void_p(ctypes.addressof(buf))
    one = ctypes.c_void_p(ctypes.addressof(buf) + 64)      # stands for any non-NULL pointer argument
    assert lib.dkv_refresh(bogus, 0) == -3
    assert lib.dkv_status(bogus, None) == -3
    assert lib.dkv_step(bogus, one, one, None, 1, 0, 1, -1, one, one, None, None) == -3
    assert lib.dkv_step_host(bogus, one, one, None, 1, 0, 1, -1, None, None) == -3
    assert lib.dkv_generate(bogus, one, one, None, 1, 0, 0, None, None) == -3
    assert lib.dkv_get_stats(bogus, ctypes.cast(one, ctypes.POINTER(B.dkv_stats))) == -3
    assert lib.dkv_get_provenance(bogus, one, None) == -3
    assert lib.dkv_get_index_maps(bogus, None, None, None, None) == -3
    assert lib.dkv_cache_slots(bogus, 0, None, None) == -3
    assert lib.dkv_profile_enable(bogus, 1) == -3
    assert lib.dkv_cache_state_bytes(bogus) == 0
    assert lib.dkv_cache_export(bogus, one, 4096, None) == -3
    assert lib.dkv_cache_import(bogus, one, 4096, None) == -3
    assert lib.dkv_cache_export(None, one, 4096, None) == -1
    assert lib.dkv_cache_destroy(bogus) == -3
    assert lib.dkv_model_destroy(bogus) == -3
    assert lib.dkv_cache_bytes(bogus, 1, 16, None) == 0
    pol = B.make_policy(B.DKV_POLICY_DECODE)
    out = ctypes.c_void_p()
    assert lib.dkv_init_cache(bogus, 1, 16, 8, ctypes.byref(pol), one, 1 << 20, None, ctypes.byref(out)) == -3
    assert b"state" in lib.dkv_strerror(-3)


def test_struct_sizes_match_the_header():
    assert ctypes.sizeof(B.dkv_model_desc) == 48
    assert ctypes.sizeof(B.dkv_policy) == 40
    assert ctypes.sizeof(B.dkv_layer_weights) == 48
    assert ctypes.sizeof(B.dkv_stats) == 56
    assert ctypes.sizeof(B.dkv_profile_entry) == 64
