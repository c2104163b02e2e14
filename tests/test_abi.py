"""The C-ABI library loads without a GPU and exports every entry point that include/mars.h
declares; the binding's table of signatures names exactly the same set.  No compute call is made."""
import ctypes
import os
import re

import pytest

from paper_2511_11373_b200 import binding, workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2511_11373_b200 import build
    build.build()
    return binding.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "mars.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mars_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported_and_bound(lib):
    names = declared_functions()
    assert "mars_decode_step" in names and "mars_prefill_chunk" in names and "mars_kv_alloc" in names
    assert "mars_model_load" in names and "mars_kv_free" in names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in mars.h but not exported"
    assert sorted(binding.SIGNATURES) == names


def test_status_strings_and_version(lib):
    assert lib.mars_version().decode().startswith("mars-rollout-b200")
    seen = {lib.mars_status_string(i).decode() for i in range(8)}
    assert len(seen) == 8 and lib.mars_status_string(99).decode() == "unknown status"


def test_workspace_and_meta_sizes_are_host_only(lib):
    cfg = binding.make_config(wl.MODEL_TINY, max_pos=512)
    small = lib.mars_workspace_bytes(ctypes.byref(cfg), 4, 0)
    big = lib.mars_workspace_bytes(ctypes.byref(cfg), 64, 256)
    assert 0 < small < big and small % 256 == 0
    assert lib.mars_workspace_bytes(ctypes.byref(cfg), 0, 0) == 0
    bad = binding.make_config(dict(wl.MODEL_TINY, head_dim=48), max_pos=512)
    assert lib.mars_workspace_bytes(ctypes.byref(bad), 4, 0) == 0          # unsupported shape
    assert lib.mars_kv_meta_bytes(4, 13) == 256 and lib.mars_kv_meta_bytes(0, 1) == 0
    full = binding.make_config(wl.MODEL_FULL, max_pos=16384 + 256)
    ws = lib.mars_workspace_bytes(ctypes.byref(full), 64, 0)
    assert 64 * 151936 * 4 < ws < 2 << 30


def test_expert_inter_beyond_the_down_kernels_shared_memory_is_unsupported(lib):
    """The streaming down kernel stages (hi, lo) activation rows of expert_inter elements in shared
    memory; a size that cannot fit is refused up front, not in mid-step after cache rows were written."""
    ok = binding.make_config(dict(wl.MODEL_TINY, expert_inter=3136), max_pos=512)
    assert lib.mars_workspace_bytes(ctypes.byref(ok), 4, 0) > 0
    big = binding.make_config(dict(wl.MODEL_TINY, expert_inter=3200), max_pos=512)
    assert lib.mars_workspace_bytes(ctypes.byref(big), 4, 0) == 0
    fake = ctypes.c_void_p(256)                               # never dereferenced: the shape is checked first
    layer = binding.mars_layer_t(*[256] * len(binding.LAYER_FIELDS))
    w = binding.mars_weights_t(fake, fake, fake, ctypes.pointer(layer))
    out = ctypes.c_void_p()
    assert lib.mars_model_load(ctypes.byref(big), ctypes.byref(w), fake, 1 << 30, 4, 0, ctypes.byref(out)) == 2
    assert not out.value


def test_null_and_bad_arguments_are_rejected_without_a_device(lib):
    assert lib.mars_model_free(None) == 6
    assert lib.mars_kv_free(None) == 6
    assert lib.mars_kv_seq_len(None, 0) == -1
    assert lib.mars_poll_status(None) == 6
    assert lib.mars_debug_bounded_wait(None, None, 0) == 6
    out = ctypes.c_void_p()
    cfg = binding.make_config(wl.MODEL_TINY, max_pos=512)
    assert lib.mars_model_load(ctypes.byref(cfg), None, None, 0, 4, 0, ctypes.byref(out)) == 1
    assert lib.mars_decode_step(None, None, None, 1, None, None, None, None, None, None) == 6


def test_product_path_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2511_11373_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text and "mars_oracle" not in text, f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2511_11373_b200" not in text and "libmars.so" not in text, f
