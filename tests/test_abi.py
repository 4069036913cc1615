"""CPU-only checks of the C-ABI boundary: the library builds, loads, exports every function the
header declares, sizes its buffers sanely and rejects bad configurations.  No kernel is launched."""
import ctypes as C
import os
import re

import pytest

import paper_2509_24007_b200 as pk
from paper_2509_24007_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return pk.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "sdlm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sdlm_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_function_is_exported(lib):
    names = _declared_functions()
    assert {"sdlm_block_attn", "sdlm_lmhead_confidence", "sdlm_accept_commit", "sdlm_kv_pages"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in sdlm.h but not exported"
    assert sorted(binding.EXPORTED) == [n for n in names]


def _cfg(**kw):
    base = dict(n_q_heads=16, n_kv_heads=2, head_dim=128, hidden=2048, vocab=151936, num_pages=2112,
                max_batch=32, max_pages_per_seq=70, max_block=8)
    base.update(kw)
    return pk.SdlmConfig(**base).to_c()


def test_buffer_sizes(lib):
    c = _cfg()
    assert lib.sdlm_pool_bytes(C.byref(c)) == 2112 * 2 * 2 * 64 * 128 * 2      # pages x heads x K|V x tokens x d x bf16
    ws = lib.sdlm_workspace_bytes(C.byref(c))
    assert 1 << 20 < ws < 1 << 28 and ws % 256 == 0


@pytest.mark.parametrize("kw", [dict(head_dim=96), dict(n_kv_heads=3), dict(hidden=2052), dict(page_size=32),
                                dict(max_block=9), dict(max_block=0), dict(n_q_heads=32, n_kv_heads=2, max_block=8),
                                dict(max_batch=0), dict(num_pages=0), dict(vocab=0), dict(softmax_scale=-1.0)])
def test_invalid_configurations_are_rejected(lib, kw):
    c = _cfg(**kw)
    assert lib.sdlm_pool_bytes(C.byref(c)) == 0
    assert lib.sdlm_workspace_bytes(C.byref(c)) == 0


def test_null_and_no_device_paths_return_codes(lib):
    import torch
    out = C.c_void_p()
    c = _cfg()
    assert lib.sdlm_create(None, None, 0, None, 0, C.byref(out)) == 1          # INVALID_ARG
    assert lib.sdlm_pool_bytes(None) == 0
    assert lib.sdlm_status_str(4) == b"KV page pool exhausted"
    assert lib.sdlm_block_attn(None, 1, 1, None, None, None, None, None, None) == 1
    assert lib.sdlm_lmhead_confidence(None, 1, None, None, None, None, None, None, None, None) == 1
    assert lib.sdlm_accept_commit(None, 1, 1, None, 0.5, 0, None, None, None, None, None, None, None, None) == 1
    assert lib.sdlm_kv_pages(None, 3, None, None, None) == 1
    assert lib.sdlm_launch_count(None) == 0
    lib.sdlm_destroy(None)
    if not torch.cuda.is_available():
        # fake but aligned pointers: creation must fail on the missing device, not touch memory
        assert lib.sdlm_create(C.byref(c), 1 << 20, 1 << 40, 1 << 20, 1 << 40, C.byref(out)) == 5   # CUDA
        with pytest.raises(pk.SdlmError):
            pk.Sdlm(pk.SdlmConfig(4, 2, 64, 256, 1024, 8, 1, 4))


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2509_24007_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f"{f} refers to the oracle"
