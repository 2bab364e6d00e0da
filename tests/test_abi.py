"""Host-side checks of the C ABI that need no GPU: the library builds, loads,
and exports every symbol include/kb.h declares; sizes and status strings."""
import ctypes
import os
import re

import pytest

from paper_2511_18868_b200 import build as kb_build
from paper_2511_18868_b200 import kb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    kb_build.build_lib()
    return kb.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "kb.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kb_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 25
    assert sorted(kb.EXPORTS) == names
    for n in names:
        assert getattr(lib, n) is not None


def test_status_strings(lib):
    assert lib.kb_status_string(0) == b"KB_OK"
    assert lib.kb_status_string(3) == b"KB_ERR_WORKSPACE"
    assert lib.kb_status_string(99) == b"KB_ERR_UNKNOWN"


def test_workspace_sizes_are_host_only_and_monotone(lib):
    out = ctypes.c_size_t()
    assert lib.kb_workspace_bytes(1, 1024, 32, 16, 8, ctypes.byref(out)) == 0
    small = out.value
    assert lib.kb_workspace_bytes(4, 1 << 20, 128, 1024, 8, ctypes.byref(out)) == 0
    assert out.value > small > 0
    assert lib.kb_workspace_bytes(-1, 1, 1, 1, 1, ctypes.byref(out)) == 1
    assert lib.kb_workspace_bytes(1, 1, 1, 1, 1, None) == 1
    assert lib.kb_step_workspace_bytes(1, 256, 16, 8, 8, 3, ctypes.byref(out)) == 0
    # staging area: at least the inputs and outputs of the step
    assert out.value > 256 * 16 * 4 + 2 * 256 * 8 * 4


def test_null_context_is_rejected(lib):
    assert lib.kb_normalize(None, 1, 1, 4, None, None, None, None) == 1
    assert lib.kb_set_workspace(None, None, 0) == 1
    assert lib.kb_bandit_step(None, None) == 1


def test_struct_layout_matches_header():
    # 7 ints + float + 5-word params + 32 pointers (13 inputs, 17 outputs, 2 for the expanding frontier), pointer-aligned
    assert ctypes.sizeof(kb.ScoreParams) == 20
    assert ctypes.sizeof(kb.StepArgs) == 56 + 8 * 32
    assert len(kb._STEP_IN) == 13 and len(kb._STEP_OUT) == 17


def test_device_status_word_maps_to_a_status(lib):
    """What a synchronising entry point returns for a device status word (no device needed: the mapping
    is a pure host function).  Timeout bits win over contract bits; contract bits count only where asked."""
    f = lib.kb_status_of_device_word
    assert f(0, 0) == 0 and f(0, 1) == 0
    assert f(0x100, 0) == 5 and f(0x200, 0) == 5 and f(0x300, 1) == 5
    assert lib.kb_status_string(f(0x100, 0)) == b"KB_ERR_TIMEOUT"
    for bit in (1, 2, 4, 7):
        assert f(bit, 0) == 0                       # kb_get_device_status leaves these to the caller
        assert f(bit, 1) == 1                       # kb_bandit_step_host reports them
        assert f(bit | 0x200, 1) == 5
    assert lib.kb_clear_device_status(None) == 1
    assert lib.kb_cluster_update_noalloc_status(None, None) == 1
