"""The C-ABI library builds, loads without a GPU and exports every symbol mrp.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(inc, fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        for m in re.finditer(r"\b(mrp_[a-z0-9_]+)\s*\(", text):
            names.add(m.group(1))
    return names


def test_library_builds_loads_and_exports_declared_symbols():
    from paper_2605_18817_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    names = declared_functions()
    assert {"mrp_create", "mrp_draft", "mrp_reveal_remask", "mrp_verify", "mrp_destroy"} <= names
    for n in names:
        assert hasattr(lib, n), n


def test_binding_mirrors_the_abi_names_and_status_strings():
    from paper_2605_18817_b200 import binding
    for n in ("mrp_create", "mrp_draft", "mrp_reveal_remask", "mrp_verify", "mrp_destroy"):
        assert callable(getattr(binding, n))
    assert binding.lib.mrp_status_string(0) == b"ok"
    assert binding.lib.mrp_status_string(1) == b"invalid argument"


def test_workspace_bytes_rejects_bad_configs_and_grows_with_rows():
    from paper_2605_18817_b200 import binding
    good = binding.mrp_config(256, 512, 4096, 3, 4, 1, 4, binding.MRP_F32, 1e-6, 0, 0)
    n1 = binding.mrp_workspace_bytes(good)
    assert n1 > 0
    big = binding.mrp_config(256, 512, 4096, 3, 64, 16, 4, binding.MRP_F32, 1e-6, 0, 0)
    assert binding.mrp_workspace_bytes(big) > n1
    for bad in (binding.mrp_config(0, 512, 4096, 3, 4, 1, 4, 0, 1e-6, 0, 0),
                binding.mrp_config(256, 512, 4096, 3, 4, 1, 4, 7, 1e-6, 0, 0),
                binding.mrp_config(256, 512, 4096, -1, 4, 1, 4, 0, 1e-6, 0, 0)):
        assert binding.mrp_workspace_bytes(bad) == 0


def test_null_arguments_are_rejected_on_the_host():
    from paper_2605_18817_b200 import binding
    lib = binding.lib
    h = ctypes.c_void_p()
    assert lib.mrp_create(None, None, None, None, 0, ctypes.byref(h)) == 1
    assert lib.mrp_draft(None, None, None, None, 1, 1, None, None) == 1
    assert lib.mrp_verify(None, None, None, None, 1, 1, 0, None, None, None) == 1
    assert lib.mrp_draft_from_hidden(None, None, None, None, 1, 1, None, None) == 1
    assert lib.mrp_commit(None, None, None, 1, 1, 0, None, None) == 1
    assert lib.mrp_set_logits0_event(None, None) == 1
    lib.mrp_destroy(None)


def test_product_path_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2605_18817_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, fn)).read()
                assert "import oracle" not in text and "from oracle" not in text, fn
                assert "mrp_oracle" not in text, fn
