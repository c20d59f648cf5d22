"""CPU-side checks of the C ABI: the library builds, loads, and exports every entry point that
include/swimba.h declares; host-side validation works without a device."""
import ctypes
import os
import re

import pytest
import torch

from paper_2603_06938_b200 import binding as sb
from paper_2603_06938_b200 import build as sbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "swimba.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(swimba_[a-z_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = sbuild.build()
    assert os.path.exists(path)
    L = ctypes.CDLL(path)
    names = declared_symbols()
    assert len(names) >= 10
    for n in names:
        assert hasattr(L, n), f"{n} declared in swimba.h but not exported"
    assert sorted(sb.EXPORTS) == names


def test_null_arguments_are_rejected_without_a_device():
    L = sb.lib()
    assert L.swimba_create(None, None) == sb.ERR_NULL_ARG
    assert L.swimba_status(None) == sb.ERR_NULL_ARG
    assert L.swimba_workspace_bytes(None, 1, 1) == 0
    assert L.swimba_forward(None, None, None, None, None, None, 1, 1, None, None, None, None, None,
                            0, None) == sb.ERR_NULL_ARG
    L.swimba_destroy(None)


def test_bad_config_is_rejected_before_touching_the_device():
    with pytest.raises(sb.SwimbaError) as e:
        sb.swimba_create(64, 4, 64, 128, 1, 4, 9, 128, sb.DTYPE_BF16)     # k > E
    assert e.value.code == sb.ERR_BAD_CONFIG


@pytest.mark.skipif(torch.cuda.is_available(), reason="only meaningful without a device")
def test_create_without_a_device_fails_loudly():
    with pytest.raises(sb.SwimbaError) as e:
        sb.swimba_create(64, 4, 64, 128, 1, 4, 2, 128, sb.DTYPE_BF16)
    assert e.value.code == sb.ERR_CUDA
