"""The C-ABI library builds, loads and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

from paper_2609_20744_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "vdn_vda.h")


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vdn_vda_[a-z_]+)\s*\(", text)))


def test_header_declares_the_north_star_entry_points():
    names = declared_functions()
    for n in ("vdn_vda_create", "vdn_vda_forward", "vdn_vda_destroy"):
        assert n in names


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), f"{n} declared in the header but not exported"
    assert set(names) == set(binding.EXPORTS)


def test_header_is_plain_c(tmp_path):
    src = tmp_path / "t.c"
    src.write_text('#include "vdn_vda.h"\nint main(void){ vdn_vda_config c; c.struct_size = sizeof c; return (int)c.struct_size == 0; }\n')
    rc = os.system(f"gcc -std=c99 -Wall -Werror -I{os.path.join(ROOT, 'include')} -c {src} -o {tmp_path / 't.o'}")
    assert rc == 0


def test_host_side_argument_errors_without_touching_a_gpu(lib):
    h = ctypes.c_void_p()
    assert lib.vdn_vda_create(None, ctypes.byref(h)) == 1
    bad = binding.VdnConfig(4, binding.VDN_BF16, 128, 1e-6, 0, 0)           # wrong struct_size
    assert lib.vdn_vda_create(ctypes.byref(bad), ctypes.byref(h)) == 1
    bad = binding.VdnConfig(ctypes.sizeof(binding.VdnConfig), 7, 128, 1e-6, 0, 0)   # unknown dtype
    assert lib.vdn_vda_create(ctypes.byref(bad), ctypes.byref(h)) == 1
    bad = binding.VdnConfig(ctypes.sizeof(binding.VdnConfig), binding.VDN_BF16, 96, 1e-6, 0, 0)
    assert lib.vdn_vda_create(ctypes.byref(bad), ctypes.byref(h)) == 2        # unsupported d
    assert h.value is None
    assert lib.vdn_vda_status(None) == 1
    assert lib.vdn_vda_destroy(None) == 1
    assert lib.vdn_vda_last_error(None) == b"null handle"
    assert lib.vdn_vda_workspace_bytes(None, 1, 1, 1, 1, 64) == 0


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(FileNotFoundError):
        binding.load_library(str(tmp_path / "nope.so"))
