"""CPU-only checks of the C-ABI boundary: the library loads, exports every symbol the
header declares, the binding mirrors the header, argument validation rejects bad calls
before any CUDA work, and the dispatcher's choices are pure functions of the shape."""
import ctypes
import os
import re

import pytest

import paper_2603_21331_b200 as ak
from paper_2603_21331_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _header_functions():
    text = open(os.path.join(ROOT, "include", "ak.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ak_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _header_functions()
    assert {"ak_rmsnorm_fwd", "ak_softmax_fwd", "ak_xent_fwd"} <= set(names)
    l = ak.lib()
    for n in names:
        assert hasattr(l, n), f"{n} declared in ak.h but not exported"
    assert sorted(binding.SIGNATURES) == names, "binding and header disagree"
    assert ak.ak_version() >= 100


def test_status_strings():
    seen = {ak.ak_status_string(s) for s in range(7)}
    assert len(seen) == 7 and ak.ak_status_string(0) == "ok"
    assert ak.ak_status_string(99) == "unknown status"


def test_validation_rejects_before_any_cuda_call():
    l = ak.lib()
    P = 0x1000  # fake, never dereferenced: every call below must fail validation first
    assert l.ak_rmsnorm_fwd(None, P, P, 1, 8, 1e-6, None) == 1
    assert l.ak_rmsnorm_fwd(P, None, P, 1, 8, 1e-6, None) == 1
    assert l.ak_rmsnorm_fwd(P, P, None, 1, 8, 1e-6, None) == 1
    assert l.ak_rmsnorm_fwd(P, P, P, -1, 8, 1e-6, None) == 2
    assert l.ak_rmsnorm_fwd(P, P, P, 1, 0, 1e-6, None) == 2
    assert l.ak_rmsnorm_fwd(P + 1, P, P, 1, 8, 1e-6, None) == 3
    assert l.ak_rmsnorm_fwd(P, P, P, 1, 8, -1.0, None) == 4
    assert l.ak_rmsnorm_fwd(P, P, P, 1, 8, float("nan"), None) == 4
    assert l.ak_rmsnorm_fwd(P, P, P, 1, 8, float("inf"), None) == 4
    assert l.ak_rmsnorm_fwd_path(P, P, P, 1, 8, 1e-6, None, 9) == 4
    assert l.ak_rmsnorm_fwd(P, P, P, 0, 8, 1e-6, None) == 0          # rows == 0: nothing to do
    assert l.ak_rmsnorm_fwd(P, P, P, 1 << 40, 1 << 40, 1e-6, None) == 2
    assert l.ak_layernorm_fwd(None, P, P, P, 1, 8, 1e-5, None) == 1
    assert l.ak_layernorm_fwd(P, None, P, P, 1, 8, 1e-5, None) == 1
    assert l.ak_layernorm_fwd(P, P, None, P, 1, 8, 1e-5, None) == 1
    assert l.ak_layernorm_fwd(P, P, P, None, 1, 8, 1e-5, None) == 1
    assert l.ak_layernorm_fwd(P, P, P, P, 1, 0, 1e-5, None) == 2
    assert l.ak_layernorm_fwd(P, P, P + 1, P, 1, 8, 1e-5, None) == 3
    assert l.ak_layernorm_fwd(P, P, P, P, 1, 8, -1e-5, None) == 4
    assert l.ak_layernorm_fwd_path(P, P, P, P, 1, 8, 1e-5, None, 6) == 4
    assert l.ak_layernorm_fwd_path(P, P, P, P, 1, 8, 1e-5, None, 5) == 2          # a cluster needs two vectors per row
    assert l.ak_layernorm_fwd(P, P, P, P, 0, 8, 1e-5, None) == 0
    assert l.ak_rowsum_fwd(None, P, 1, 8, None) == 1
    assert l.ak_rowsum_fwd(P, None, 1, 8, None) == 1
    assert l.ak_rowsum_fwd(P, P, 1, 0, None) == 2
    assert l.ak_rowsum_fwd(P + 1, P, 1, 8, None) == 3
    assert l.ak_rowsum_fwd(P, P + 2, 1, 8, None) == 3                # fp32 sums need 4 B
    assert l.ak_rowsum_fwd(P, P, 0, 8, None) == 0
    # element-type variants: unknown dtype, fp32 alignment
    assert l.ak_rmsnorm_fwd_dt(P, P, P, 1, 8, 1e-6, 7, None, 0) == 4
    assert l.ak_rmsnorm_fwd_dt(P + 2, P, P, 1, 8, 1e-6, 2, None, 0) == 3     # fp32 needs 4 B
    assert l.ak_softmax_fwd_dt(P, P + 2, 1, 8, 2, None, 0) == 3
    assert l.ak_softmax_fwd_dt(P, P, 1, 8, -1, None, 0) == 4
    assert l.ak_xent_fwd_dt(P + 2, P, -100, P, P, 1, 8, 2, None, 0, 0) == 3
    assert l.ak_xent_fwd_dt(P, P, -100, P, P, 1, 8, 3, None, 0, 0) == 4
    assert l.ak_choose_path_dt(0, 8192, 4096, 1, 2) == ak.AK_PATH_CTA       # 16 KiB fp32 rows
    assert l.ak_choose_path_dt(0, 8192, 1024, 1, 2) == ak.AK_PATH_WARP
    assert l.ak_choose_path_dt(0, 8192, 1022, 1, 2) == ak.AK_PATH_GENERIC   # 4088 B: not a multiple of 16
    assert l.ak_choose_path_dt(1, 8192, 8192, 1, 2) == ak.AK_PATH_SMEM      # 32 KiB fp32 softmax rows
    assert l.ak_choose_path_dt(1, 8192, 8192, 1, 1) == ak.AK_PATH_CTA
    assert l.ak_choose_path_dt(3, 1, 8, 1, 0) == -1 and l.ak_choose_path_dt(0, 1, 8, 1, 9) == -1
    assert l.ak_choose_path_dt(2, 8192, 4096, 1, 2) == ak.AK_PATH_CTA and l.ak_choose_path_dt(2, 8192, 4096, 1, 0) == ak.AK_PATH_CTA
    assert l.ak_layernorm_fwd_dt(P, P, P + 2, P, 1, 8, 1e-5, 2, None, 0) == 3
    assert l.ak_layernorm_fwd_dt(P, P, P, P, 1, 8, 1e-5, 5, None, 0) == 4
    assert l.ak_rowsum_fwd_dt(P + 2, P, 1, 8, 2, None) == 3 and l.ak_rowsum_fwd_dt(P, P, 1, 8, 4, None) == 4
    # vocabulary-parallel cross-entropy
    assert l.ak_xent_vp_partial_bytes(10, 3) == 10 * 4 * 8 and l.ak_xent_vp_partial_bytes(0, 3) == 0
    assert l.ak_xent_vp_nsplit(4096, 16032) == 1 and l.ak_xent_vp_nsplit(16, 16032) == 1
    assert l.ak_xent_vp_nsplit(16, 64128) == 4                  # slices of at most 16384 elements
    assert l.ak_xent_vp_partial(None, P, -100, 0, 64, P, 1, 32, 1, 0, None) == 1
    assert l.ak_xent_vp_partial(P, P, -100, 40, 64, P, 1, 32, 1, 0, None) == 2   # shard sticks out of the vocabulary
    assert l.ak_xent_vp_partial(P, P, -100, 0, 64, P, 1, 0, 1, 0, None) == 2     # empty shard
    assert l.ak_xent_vp_partial(P, P, -100, 0, 64, P, 1, 32, 0, 0, None) == 4
    assert l.ak_xent_vp_partial(P, P, -100, 0, 64, P + 4, 1, 32, 1, 0, None) == 3
    assert l.ak_xent_vp_merge(None, 2, 1, P, -100, 64, P, P, 1, None) == 1
    assert l.ak_xent_vp_merge(P, 0, 1, P, -100, 64, P, P, 1, None) == 4
    assert l.ak_xent_vp_merge(P, 2, 65, P, -100, 64, P, P, 1, None) == 4
    assert l.ak_softmax_fwd(None, P, 1, 8, None) == 1
    assert l.ak_softmax_fwd(P, P, 1, -3, None) == 2
    assert l.ak_softmax_fwd(P, P + 1, 1, 8, None) == 3
    assert l.ak_softmax_fwd_path(P, P, 1, 8, None, -1) == 4
    assert l.ak_softmax_fwd(P, P, 0, 8, None) == 0
    assert l.ak_xent_fwd(None, P, -100, P, P, 1, 8, None) == 1
    assert l.ak_xent_fwd(P, None, -100, P, P, 1, 8, None) == 1
    assert l.ak_xent_fwd(P, P, -100, None, P, 1, 8, None) == 1
    assert l.ak_xent_fwd(P, P, -100, P, P, 1, 0, None) == 2
    assert l.ak_xent_fwd(P, P + 4, -100, P, P, 1, 8, None) == 3      # int64 targets need 8 B
    assert l.ak_xent_fwd(P, P, -100, P + 2, P, 1, 8, None) == 3      # fp32 losses need 4 B
    assert l.ak_xent_fwd_path(P, P, -100, P, P, 1, 8, None, 5, 0) == 4
    assert l.ak_xent_fwd_path(P, P, -100, P, P, 1, 8, None, 2, 65) == 4
    # workspace variant: too small / missing workspace for a shape that splits
    need = ak.ak_xent_workspace_bytes(16, 128256)
    assert need > 0
    assert l.ak_xent_fwd_ws(P, P, -100, P, P, 16, 128256, None, 0, None) == 1
    assert l.ak_xent_fwd_ws(P, P, -100, P, P, 16, 128256, P, need - 1, None) == 6
    assert l.ak_xent_fwd_ws(P, P, -100, P, P, 16, 128256, P + 4, need, None) == 3
    # host variants validate the same way
    assert l.ak_rmsnorm_fwd_host(None, P, P, 1, 8, 1e-6) == 1
    assert l.ak_softmax_fwd_host(P, P, -1, 8) == 2
    assert l.ak_xent_fwd_host(P, P + 4, -100, P, P, 1, 8) == 3


def test_dispatch_is_a_pure_function_of_shape_and_alignment():
    assert ak.ak_rmsnorm_choose_path(8192, 1024, True) == ak.AK_PATH_WARP
    assert ak.ak_rmsnorm_choose_path(8192, 4096, True) == ak.AK_PATH_CTA
    assert ak.ak_rmsnorm_choose_path(8192, 16384, True) == ak.AK_PATH_CTA
    assert ak.ak_rmsnorm_choose_path(8192, 32768, True) == ak.AK_PATH_CTA
    assert ak.ak_rmsnorm_choose_path(8192, 32776, True) == ak.AK_PATH_CLUSTER    # longer than 64 KiB: split over a cluster
    assert ak.ak_layernorm_choose_path(8192, 32768, True) == ak.AK_PATH_CTA
    assert ak.ak_layernorm_choose_path(8192, 40960, True) == ak.AK_PATH_CLUSTER
    assert ak.ak_rmsnorm_choose_path(8192, 4099, True) == ak.AK_PATH_GENERIC
    assert ak.ak_rmsnorm_choose_path(8192, 4096, False) == ak.AK_PATH_GENERIC
    assert ak.ak_rmsnorm_choose_path(8192, 65536, True) == ak.AK_PATH_CLUSTER
    assert ak.ak_rmsnorm_choose_path(8192, 131072, True) == ak.AK_PATH_CLUSTER   # 256 KiB rows: four to eight CTAs' shared memory
    assert ak.ak_rmsnorm_choose_path(8192, 917504, True) == ak.AK_PATH_CLUSTER   # 8 x 224 KiB, the longest
    assert ak.ak_rmsnorm_choose_path(8192, 917512, True) == ak.AK_PATH_CLUSTER   # beyond that: streamed by the cluster
    assert ak.ak_rmsnorm_choose_path(64, 16384, True) == ak.AK_PATH_CLUSTER      # few rows of 32 KiB or more
    assert ak.ak_rmsnorm_choose_path(65, 16384, True) == ak.AK_PATH_CTA
    assert ak.ak_rmsnorm_choose_path(64, 8192, True) == ak.AK_PATH_CTA
    assert ak.ak_softmax_choose_path(16384, 16384, True) == ak.AK_PATH_SMEM
    assert ak.ak_softmax_choose_path(16, 128256, True) == ak.AK_PATH_CLUSTER
    assert ak.ak_softmax_choose_path(16384, 512, True) == ak.AK_PATH_WARP
    assert ak.ak_softmax_choose_path(16384, 8192, True) == ak.AK_PATH_CTA
    assert ak.ak_softmax_choose_path(16384, 32768, True) == ak.AK_PATH_SMEM
    assert ak.ak_softmax_choose_path(16384, 32776, True) == ak.AK_PATH_CLUSTER   # longer than 64 KiB
    assert ak.ak_softmax_choose_path(16384, 128257, True) == ak.AK_PATH_GENERIC
    for rows, V in ((4096, 32000), (4096, 128256), (16384, 128256)):
        assert ak.ak_xent_choose_path(rows, V) == (ak.AK_XENT_ROW, 1)
        assert ak.ak_xent_workspace_bytes(rows, V) == 0
    path, ns = ak.ak_xent_choose_path(16, 128256)
    assert path == ak.AK_XENT_SPLIT and 2 <= ns <= 64
    assert ak.ak_xent_workspace_bytes(16, 128256) == 16 * ns * 8
    assert ak.ak_xent_choose_path(1, 128256)[1] == 8             # slices of at most 16384 elements
    # the split rules are stated in SMs of the current device (148 when none can be queried)
    sms = ak.ak_sm_count()
    assert sms >= 1
    assert ak.ak_xent_choose_path(4 * sms - 1, 128256)[0] == ak.AK_XENT_SPLIT
    assert ak.ak_xent_choose_path(4 * sms, 128256) == (ak.AK_XENT_ROW, 1)
    assert ak.ak_xent_choose_path(16, 1000) == (ak.AK_XENT_ROW, 1)  # short rows never split
    # repeated queries agree (no hidden state)
    assert all(ak.ak_xent_choose_path(16, 128256) == (path, ns) for _ in range(3))


def test_binding_refuses_cpu_tensors_instead_of_falling_back():
    import torch
    x = torch.zeros((2, 8), dtype=torch.bfloat16)
    with pytest.raises(TypeError):
        ak.ak_rmsnorm_fwd(x, torch.ones(8, dtype=torch.bfloat16))
    with pytest.raises(TypeError):
        ak.ak_softmax_fwd(x)
    with pytest.raises(TypeError):
        ak.ak_xent_fwd(x, torch.zeros(2, dtype=torch.int64))


def test_product_does_not_import_the_checker():
    pkg = os.path.join(ROOT, "paper_2603_21331_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f"{f} mentions the checker"
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2603_21331_b200" not in text and "libak" not in text


def test_calls_act_on_the_tensors_device():
    """The library launches on the current CUDA device, so the binding makes the tensors' device
    current around a call and refuses a call whose tensors sit on different devices.  Checked
    here with stand-ins for tensors (no GPU needed): only `.device.index` is looked at."""
    import types
    from unittest import mock

    def on(index):
        return types.SimpleNamespace(device=types.SimpleNamespace(index=index))

    with pytest.raises(ValueError):
        binding._on_device_of(on(0), on(1))
    seen = []
    with mock.patch.object(binding.torch.cuda, "current_device", return_value=0), \
            mock.patch.object(binding.torch.cuda, "set_device", side_effect=seen.append):
        with binding._on_device_of(on(0), None, on(0)):
            pass
        assert seen == []                      # already current: nothing is switched
        with binding._on_device_of(on(1), on(1)):
            assert seen == [1]
        assert seen == [1, 0]                  # and put back afterwards


def test_wait_timeout_flags_have_a_host_reader():
    # without a device the flags cannot be read (-1); with one, no wait has ever given up (0)
    assert ak.ak_wait_timeouts() in (-1, 0)


def test_kernels_compile_without_spills():
    """Every kernel of the library keeps everything in registers: the compiler's own report
    (written next to the library by its build) shows no spill stores or loads for any entry
    function.  Skipped when the library was built elsewhere and the report is not at hand."""
    log = os.path.join(ROOT, "paper_2603_21331_b200", "build", "ptxas.log")
    if not os.path.exists(log):
        pytest.skip("no compiler report beside the library")
    text = open(log).read()
    entries = re.findall(r"Compiling entry function '(\S+)' for 'sm_100a'\n.*?\n\s+(\d+) bytes stack frame, "
                         r"(\d+) bytes spill stores, (\d+) bytes spill loads", text)
    families = ("xent_row_kernel", "xent_split_kernel", "xent_finish_kernel", "xent_vp_partial_kernel",
                "xent_vp_merge_kernel", "rmsnorm_reg_kernel", "softmax_reg_kernel", "softmax_smem_kernel",
                "layernorm_reg_kernel", "rowsum_kernel", "rope_vec_kernel", "_cluster_kernel", "_stage_kernel",
                "_regp_kernel")
    seen = set()
    for name, _, stores, loads in entries:
        assert int(stores) == 0 and int(loads) == 0, f"{name} spills {stores} / {loads} bytes"
        seen.update(f for f in families if f in name)
    assert seen == set(families), f"families missing from the report: {set(families) - seen}"
    assert len(entries) >= 300   # every instantiation was looked at
