"""Host-side checks of the C-ABI library that need no GPU: it builds for sm_100a, loads,
exports every function include/optiml.h declares, and its host logic (strings, version,
argument checks that run before any CUDA call) behaves."""
import ctypes
import os
import re

import pytest
import torch

from paper_2602_12305_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()          # nvcc cross-compiles without a GPU; no-op when fresh
    return binding.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "optiml.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(optiml_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert "optiml_gemm_epilogue" in names and len(names) >= 10
    for n in names:
        assert hasattr(lib, n), f"{n} declared in optiml.h but not exported"
    assert sorted(binding.EXPORTS) == names, "binding.EXPORTS and optiml.h disagree"


def test_header_compiles_as_plain_c(tmp_path):
    import subprocess
    src = tmp_path / "t.c"
    src.write_text('#include "optiml.h"\nint main(void){return (int)OPTIML_VARIANT_COUNT - 7;}\n')
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), "-c", str(src),
                    "-o", str(tmp_path / "t.o")], check=True)


def test_strings_and_version(lib):
    assert binding.version() >= 100
    assert binding.status_string(binding.OK) == "ok"
    seen = {binding.status_string(c) for c in range(8)}
    assert len(seen) == 8 and "unknown status" not in seen
    assert binding.status_string(99) == "unknown status"
    names = [binding.variant_name(v) for v in range(binding.VARIANT_COUNT)]
    assert len(set(names)) == binding.VARIANT_COUNT and "unknown" not in names
    assert binding.variant_name(binding.VARIANT_AUTO) == "auto" and binding.variant_name(42) == "unknown"


def test_null_arguments_are_rejected_before_any_cuda_call(lib):
    assert lib.optiml_create(None, 0) == binding.ERR_INVALID_ARG
    assert lib.optiml_destroy(None) == binding.OK
    assert lib.optiml_gemm_epilogue(None, 16, 16, None, 16, 1, 1, 1, 0, 0, None) == binding.ERR_INVALID_ARG
    assert lib.optiml_gemm_epilogue_host(None, 16, 16, None, 16, 1, 1, 1, 0, 0, None) == binding.ERR_INVALID_ARG
    assert lib.optiml_get_last_status(None) == binding.ERR_INVALID_ARG
    assert lib.optiml_force_variant(None, 0) == binding.ERR_INVALID_ARG
    assert lib.optiml_select_variant(None, 1, 1, 1, 0) == -1
    assert lib.optiml_launch_count(None) == -1
    assert lib.optiml_set_option(None, 0, 1) == binding.ERR_INVALID_ARG
    assert lib.optiml_get_option(None, 0) == -1
    assert lib.optiml_selftest_timeout(None, 1000, None) == binding.ERR_INVALID_ARG
    assert lib.optiml_reduce_f32(None, 0, 16, None, 1, 16, None) == binding.ERR_INVALID_ARG
    assert lib.optiml_mhsa(None, 16, 16, 16, 16, 1, 1, 1, 1, None) == binding.ERR_INVALID_ARG


def test_alloc_hook_can_be_set_and_removed_without_a_gpu(lib):
    calls = []
    cb = binding.ALLOC_HOOK(lambda nbytes, user: calls.append(nbytes) or 1)
    binding.set_alloc_hook(cb)
    binding.set_alloc_hook(None)
    assert calls == []                      # setting a hook allocates nothing by itself


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU behaviour")
def test_create_without_a_gpu_fails_loudly(lib):
    h = ctypes.c_void_p()
    rc = lib.optiml_create(ctypes.byref(h), 0)
    assert rc in (binding.ERR_CUDA, binding.ERR_INVALID_ARG, binding.ERR_ARCH) and not h.value
    with pytest.raises(binding.OptimlError):
        binding.Handle(0)


def test_missing_library_raises_instead_of_falling_back(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/liboptiml_gemm.so")
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.load_library()


def test_product_path_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2602_12305_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                for needle in ("import oracle", "from oracle", "oracle.", "oracle/", "gemm_epilogue_oracle"):
                    assert needle not in text, f"{f} reaches for the oracle ({needle!r})"
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2602_12305_b200" not in text and "optiml.h" not in text
