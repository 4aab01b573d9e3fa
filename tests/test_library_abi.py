"""CPU-side checks of the boundary: the library loads and exports every symbol include/marlaas.h declares,
and host-side argument validation answers with status codes without needing a GPU."""
import ctypes
import os
import re

import pytest

import paper_2605_08527_b200 as ml
from paper_2605_08527_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "marlaas.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(marlaas_[a-z_]+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib():
    from paper_2605_08527_b200 import build
    build.build()
    return B.load_library()


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert "marlaas_lora_forward" in names and "marlaas_lora_backward" in names
    assert "marlaas_adapter_pool_register" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in marlaas.h but not exported"
    assert sorted(B.EXPORTED_SYMBOLS) == names


def test_storage_bytes_and_argument_checks(lib):
    assert lib.marlaas_adapter_pool_storage_bytes(4096, 4096, 16, 32) > 2 * 32 * 16 * 4096 * 2
    assert lib.marlaas_adapter_pool_storage_bytes(4096, 4097, 16, 32) == 0      # d_out not a multiple of 8
    assert lib.marlaas_adapter_pool_storage_bytes(4096, 4096, 0, 32) == 0
    assert lib.marlaas_adapter_pool_storage_bytes(4096, 4096, 129, 32) == 0
    h = ctypes.c_void_p()
    rc = lib.marlaas_adapter_pool_create(ctypes.byref(h), 0, 512, 511, 8, 4, None, 0, None)
    assert rc == B.MARLAAS_ERR_INVALID_ARG and "multiples of 8" in B.marlaas_last_error()
    rc = lib.marlaas_adapter_pool_create(ctypes.byref(h), 0, 512, 512, 8, 4, None, 0, None)
    # without a GPU the device check answers; with one, the NULL storage does
    assert rc in (B.MARLAAS_ERR_UNSUPPORTED_DEVICE, B.MARLAAS_ERR_INVALID_ARG)
    assert lib.marlaas_lora_forward(None, 1, None, 0, None, 0, None, 0, None, None, None, 0, 0, None) == B.MARLAAS_ERR_INVALID_ARG
    assert lib.marlaas_lora_backward(None, 1, None, 0, None, 0, None, 0, None, 0, None, None, None, None, None, 0, 0,
                                     None) == B.MARLAAS_ERR_INVALID_ARG
    assert lib.marlaas_lora_workspace_bytes(None, 5) == 0
    # pools over several projections: 1 to 4 parts, each a positive multiple of 256 columns
    def widths(*w):
        return (ctypes.c_int64 * len(w))(*w)
    one = lib.marlaas_adapter_pool_storage_bytes(4096, 4096 + 1024 + 1024, 16, 32)
    seg = lib.marlaas_adapter_pool_storage_bytes_segmented(4096, 3, widths(4096, 1024, 1024), 16, 32)
    # three blocks of A rows, ONE set of B rows over the side-by-side columns: more than a plain pool of that width by
    # two blocks of A, far less than the block-diagonal form of rank 48
    assert seg == one + 2 * 32 * 16 * 4096 * 2
    assert seg < lib.marlaas_adapter_pool_storage_bytes(4096, 4096 + 1024 + 1024, 48, 32)
    assert lib.marlaas_adapter_pool_storage_bytes_segmented(4096, 2, widths(4096, 1000), 16, 32) == 0
    assert lib.marlaas_adapter_pool_storage_bytes_segmented(4096, 5, widths(256, 256, 256, 256, 256), 16, 32) == 0
    assert lib.marlaas_adapter_pool_storage_bytes_segmented(4096, 0, widths(256), 16, 32) == 0
    assert lib.marlaas_adapter_pool_storage_bytes_segmented(4096, 2, None, 16, 32) == 0
    rc = lib.marlaas_adapter_pool_create_segmented(ctypes.byref(h), 0, 512, 2, widths(256, 384), 8, 4, None, 0, None)
    assert rc == B.MARLAAS_ERR_INVALID_ARG and "multiple of 256" in B.marlaas_last_error()
    rc = lib.marlaas_adapter_pool_create_segmented(ctypes.byref(h), 0, 512, 2, widths(256, 512), 8, 4, None, 0, None)
    assert rc in (B.MARLAAS_ERR_UNSUPPORTED_DEVICE, B.MARLAAS_ERR_INVALID_ARG)
    assert lib.marlaas_adapter_pool_parts(None) == 0
    assert lib.marlaas_lora_forward_workspace_min_bytes(None, 5) == 0


def test_product_path_has_no_oracle_or_cpu_fallback():
    pkg = os.path.join(ROOT, "paper_2605_08527_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in src and "from oracle" not in src, f
                assert "marlaas_oracle" not in src, f


def test_header_is_valid_c99(tmp_path):
    # the boundary is a C ABI: the header must compile as plain C, with every flag a distinct power of two
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no gcc")
    flags = re.findall(r"\b(MARLAAS_FLAG_[A-Z_]+)\s*=\s*(\d+)u", open(os.path.join(ROOT, "include", "marlaas.h")).read())
    values = [int(v) for _, v in flags]
    assert len(flags) >= 6 and len(set(values)) == len(values) and all(v & (v - 1) == 0 for v in values)
    src = tmp_path / "h.c"
    src.write_text('#include "marlaas.h"\nint main(void) { return (int)sizeof(marlaas_segments_t) > 0 ? 0 : 1; }\n')
    r = subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-I", os.path.join(ROOT, "include"),
                        "-c", str(src), "-o", str(tmp_path / "h.o")], capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    for name, v in flags:
        assert getattr(B, name) == int(v), name
