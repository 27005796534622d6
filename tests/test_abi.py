"""The C-ABI library builds, loads without a GPU and exports everything include/dppo.h declares; its
host-only entry points (version, workspace queries, argument validation) behave as documented."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2603_04135_b200 import build
    build.build_library()
    from paper_2603_04135_b200 import binding
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "dppo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dppo_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(B):
    names = declared_functions()
    assert {"dppo_version", "dppo_last_error", "dppo_group_advantages", "dppo_prune_and_rescale",
            "dppo_pack_workspace_bytes", "dppo_pack_prompts", "dppo_grpo_loss_workspace_bytes",
            "dppo_grpo_loss_fwd_bwd", "dppo_pack_prompts_static", "dppo_pack_static_max_units",
            "dppo_history_gather", "dppo_history_scatter", "dppo_lmhead_workspace_bytes",
            "dppo_lmhead_grpo_loss", "dppo_sequence_log_ratio", "dppo_grpo_loss_kernel_choice"} <= set(names)
    for n in names:
        assert hasattr(B.lib, n), n
    assert B.version() >= 100


def test_struct_layouts_match_header(B):
    assert ctypes.sizeof(B.PruneParams) == 48
    assert ctypes.sizeof(B.PackParams) == 16 and ctypes.sizeof(B.LossKernelChoice) == 16
    assert ctypes.sizeof(B.LossParams) == 80 and B.LossParams.seq_log_ratio.offset == 72
    assert ctypes.sizeof(B.LmheadParams) == 104 and B.LmheadParams.dW_dtype.offset == 92
    assert B.LossParams.row_stride.offset == 16 and B.LossParams.eps_lo.offset == 32


def test_workspace_queries(B):
    assert B.pack_workspace_bytes(B.PackParams(256, 8192, 16, 0)) >= 2 * 256 * 4
    assert B.pack_workspace_bytes(B.PackParams(65536, 8192, 16, 0)) == 2 * 65536 * 4
    big = B.pack_workspace_bytes(B.PackParams(1 << 20, 8192, 16, 0))                 # dataset-sized: the placed-bitmask too
    assert big >= 2 * (1 << 20) * 4 + (1 << 20) // 8
    assert B.pack_workspace_bytes(B.PackParams((1 << 21) + 1, 8192, 16, 0)) == 0    # above the unit limit
    n = B.grpo_loss_workspace_bytes(B.LossParams(1000, 1024, 0, 1024, 4, 0, 0.2, 0.2, 0.04, 1.0))
    assert n >= 1000 * 32 and n % 256 == 0


def test_host_validation_needs_no_device(B):
    # these return before anything is launched
    with pytest.raises(B.DppoError) as e:
        B.group_advantages(None, 4, 0, None, None)
    assert e.value.code == B.ERR_INVALID_ARG and "G=0" in str(e.value)
    with pytest.raises(B.DppoError) as e:
        B.group_advantages(None, 4, 4, None, None, std_ddof=2)
    assert e.value.code == B.ERR_INVALID_ARG
    B.group_advantages(None, 0, 4, None, None)                                       # P == 0: no-op
    prm = B.PruneParams(4, 4, 1.0, 0.5, 0, 0, 0, 0)
    with pytest.raises(B.DppoError) as e:
        B.prune_and_rescale(prm, *([None] * 15))
    assert e.value.code == B.ERR_INVALID_ARG and "[0,1)" in B.last_error()
    with pytest.raises(B.DppoError) as e:
        B.pack_prompts(B.PackParams(8, 0, 4, 0), *([None] * 9), None, 0)
    assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(B.DppoError) as e:
        B.pack_prompts(B.PackParams((1 << 21) + 1, 64, 4, 0), *([None] * 9), None, 0)
    assert e.value.code == B.ERR_BAD_SHAPE
    with pytest.raises(B.DppoError) as e:
        B.grpo_loss_fwd_bwd(B.LossParams(8, 0, 0, 0, 1, 0, 0.2, 0.2, 0.04, 1.0), *([None] * 14), 0)
    assert e.value.code == B.ERR_INVALID_ARG


def test_package_has_no_cpu_path():
    import torch
    if torch.cuda.is_available():
        pytest.skip("device present")
    from paper_2603_04135_b200.step import DppoStep
    with pytest.raises(RuntimeError):
        DppoStep(4, 4, 512, 4, 0.5, 0.5, 1024, "f32", 16)
