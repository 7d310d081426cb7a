"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

from paper_2604_15750_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = []
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            src = open(os.path.join(inc, fn)).read()
            names += re.findall(r"DC_API\s+[\w\s\*]+?\b(dc_\w+)\s*\(", src)
    return names


def test_library_exports_every_declared_symbol():
    lib = binding.load_library()
    names = _declared()
    assert {"dc_create", "dc_step", "dc_select", "dc_destroy"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(binding.EXPORTS)


def test_struct_sizes_match_the_header_layout():
    # 28 four-byte fields; two ints + nine pointers; pointer-only structs
    assert ctypes.sizeof(binding.dc_config) == 28 * 4
    assert ctypes.sizeof(binding.dc_step_in) == 8 + 12 * 8
    assert ctypes.sizeof(binding.dc_step_out) == 12 * 8
    assert ctypes.sizeof(binding.dc_weights) == 15 * 8
    assert ctypes.sizeof(binding.dc_select_out) == 3 * 8
    assert ctypes.sizeof(binding.dc_commit_in) == 8 + 5 * 8
    assert ctypes.sizeof(binding.dc_generate_in) == 8 + 3 * 8 + 16
    assert ctypes.sizeof(binding.dc_generate_out) == 4 * 8


def test_last_error_without_context_is_a_string():
    lib = binding.load_library()
    assert isinstance(lib.dc_last_error(None), bytes)


def test_create_rejects_null_arguments_without_a_gpu():
    lib = binding.load_library()
    ctx = ctypes.c_void_p()
    assert lib.dc_create(None, None, None, ctypes.byref(ctx)) == 1
    assert b"null" in lib.dc_last_error(None)
