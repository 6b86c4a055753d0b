"""The shared library loads on a machine without a GPU and exports every symbol the header
declares; struct layouts of the binding match the header (no compute is called here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "asyncflow.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2507_01663_b200 import build as b
    b.build()
    from paper_2507_01663_b200 import binding
    return binding.load_library()


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(af_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"af_pack_microbatch", "af_token_logprob", "af_grpo_advantage", "af_policy_loss",
            "af_policy_loss_backward"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    from paper_2507_01663_b200 import binding
    assert sorted(binding.EXPORTS) == names


def test_status_strings(lib):
    assert lib.af_status_string(0) == b"ok"
    for code in range(-9, 0):
        assert lib.af_status_string(code) not in (b"ok", b"unknown status")
    assert lib.af_status_string(-99) == b"unknown status"


def test_struct_layouts_match_header():
    from paper_2507_01663_b200 import binding as B
    # sizes follow from the header's field lists on LP64: pointers and int64 are 8 bytes
    assert ctypes.sizeof(B.StoreView) == 8 + 4 + 4 + 6 * 8
    assert ctypes.sizeof(B.Packed) == 8 + 4 + 4 + 7 * 8
    assert ctypes.sizeof(B.LossParams) == 20
    assert ctypes.sizeof(B.LossOut) == 32 and B.LossOut.n_tokens.offset == 24
    assert ctypes.sizeof(B.ControllerView) == 8 + 3 * 8
    assert ctypes.sizeof(B.GetResult) == 16 and B.GetResult.tokens.offset == 8
    assert ctypes.sizeof(B.WriteCols) == 8 + 2 * 4 * 8 and B.WriteCols.store.offset == 8 + 4 * 8


def test_create_without_gpu_fails_cleanly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    h = ctypes.c_void_p()
    assert lib.af_create(ctypes.byref(h), 0) == -8      # AF_ERR_UNSUPPORTED_DEVICE
    assert not h.value
    assert lib.af_create(None, 0) == -1
