"""The C-ABI library loads without a GPU and exports every symbol include/pt.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def built():
    from paper_1901_09290_b200 import build
    return build.build()


def _declared():
    src = open(os.path.join(ROOT, "include", "pt.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(pt_[a-z0-9_]+)\s*\(", src)))


def test_header_declares_the_call_set():
    names = _declared()
    for n in ("pt_conv_fwd", "pt_conv_dgrad", "pt_conv_wgrad", "pt_group_lasso_sgd_step", "pt_find_zero_groups",
              "pt_reconfigure", "pt_reconfigure_plan", "pt_create", "pt_destroy"):
        assert n in names


def test_library_exports_every_declared_symbol(built):
    L = ctypes.CDLL(built)
    for n in _declared():
        assert hasattr(L, n), n


def test_binding_covers_every_declared_symbol(built):
    from paper_1901_09290_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()
    binding.lib()
    for n in _declared():
        if n in ("pt_create", "pt_destroy", "pt_status_string", "pt_last_cuda_error", "pt_launch_count",
                 "pt_poll_device_status"):
            continue
        assert hasattr(binding, n), n


def test_status_strings(built):
    from paper_1901_09290_b200 import binding
    L = binding.lib()
    assert L.pt_status_string(0) == b"PT_OK" and L.pt_status_string(5) == b"PT_ERR_TIMEOUT"
    assert L.pt_last_cuda_error() == b""            # nothing failed on this thread yet


def test_create_without_gpu_fails_loudly(built):
    import torch
    from paper_1901_09290_b200 import binding
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(binding.PtError):
        binding.Context(0)


def test_struct_layouts_match_the_header(built):
    # sizes the C compiler gives the ABI structs (LP64): checked against the ctypes mirrors
    from paper_1901_09290_b200 import binding as B
    assert ctypes.sizeof(B.pt_conv_desc) == 14 * 4
    assert ctypes.sizeof(B.pt_layer) == 88 and B.pt_layer.sumsq_out.offset == 56
    assert ctypes.sizeof(B.pt_sgd_hparams) == 16 and ctypes.sizeof(B.pt_space) == 8
    assert ctypes.sizeof(B.pt_layer_link) == 40 and ctypes.sizeof(B.pt_graph) == 40
