"""CPU-side checks of the C-ABI boundary: the library loads, exports every symbol the header declares, sizes its
workspaces sanely and rejects bad arguments on the host before anything is launched (no GPU needed)."""
import ctypes
import os
import re

import pytest

from paper_2509_05576_b200 import build as ptq_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    path = ptq_build.build()
    from paper_2509_05576_b200 import ptq
    assert ptq.LIB_PATH == path
    return ptq.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "ptq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ptq_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = _declared()
    assert {"ptq_hessian_accumulate", "ptq_prepare_hinv", "ptq_sensitivity_order", "ptq_quantize_layer"} <= set(names)
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in ptq.h but not exported"
    from paper_2509_05576_b200 import ptq
    assert sorted(ptq.EXPORTS) == names
    assert lib.ptq_version() >= 1
    assert ptq.status_string(4) == "matrix not positive definite"


def test_workspace_sizes(lib):
    from paper_2509_05576_b200 import ptq
    for call in range(6):
        small = ptq.workspace_bytes(call, 64, 128, 1024)
        big = ptq.workspace_bytes(call, 256, 2304, 4096)
        assert 0 < small < big
        assert small % 256 == 0
    # the inverse needs two cols x cols float64 matrices
    assert 2 * 2304 * 2304 * 8 <= ptq.workspace_bytes(ptq.CALL_PREPARE_HINV, 0, 2304, 0) <= 2 * 2304 * 2304 * 8 + 2304 * 64 * 8 + 4096
    assert ptq.workspace_bytes(99, 1, 1, 1) == 0
    # largest benchmark shape stays far below the 180 GB of one GPU
    total = sum(ptq.workspace_bytes(c, 4096, 11008, 8192) for c in range(4))
    assert total < 8 * 2 ** 30


def test_bad_arguments_are_rejected_on_the_host(lib):
    from paper_2509_05576_b200 import ptq
    vp = ctypes.c_void_p
    fake = vp(4096)          # never dereferenced: argument checks come first
    odd = vp(4100)           # not 16-byte aligned
    assert lib.ptq_hessian_accumulate(None, fake, 8, 8, 8, fake, 1 << 30, fake, None) == ptq.ERR_INVALID_ARG
    assert lib.ptq_hessian_accumulate(fake, fake, 8, 16, 8, fake, 1 << 30, fake, None) == ptq.ERR_INVALID_ARG  # ldx < n
    assert lib.ptq_hessian_accumulate(odd, fake, 8, 8, 8, fake, 1 << 30, fake, None) == ptq.ERR_ALIGNMENT
    assert lib.ptq_hessian_accumulate(fake, fake, 8, 8, 8, fake, 16, fake, None) == ptq.ERR_WORKSPACE
    assert lib.ptq_hessian_accumulate_f64(fake, fake, 0, 8, 8, fake, 1 << 30, fake, None) == ptq.ERR_INVALID_ARG
    assert lib.ptq_prepare_hinv(fake, 8, 7, 0.01, fake, fake, fake, fake, 1 << 30, fake, None) == ptq.ERR_INVALID_ARG
    assert lib.ptq_prepare_hinv(fake, 8, 0, -1.0, fake, fake, fake, fake, 1 << 30, fake, None) == ptq.ERR_INVALID_ARG
    assert lib.ptq_prepare_hinv(fake, 8, 0, 0.01, fake, fake, fake, fake, 8, fake, None) == ptq.ERR_WORKSPACE
    assert lib.ptq_minmax_grid(fake, 4, 8, 8, 9, fake, fake, fake, None) == ptq.ERR_INVALID_ARG      # bits > 8
    assert lib.ptq_minmax_grid(fake, 4, 8, 4, 4, fake, fake, fake, None) == ptq.ERR_INVALID_ARG      # ldw < cols
    assert lib.ptq_sensitivity_order(fake, 4, 8, 8, None, fake, fake, 4, 0, fake, fake, fake, 1 << 30, fake,
                                     None) == ptq.ERR_INVALID_ARG                                   # QERR needs diag
    assert lib.ptq_sensitivity_order(fake, 4, 8, 8, fake, fake, fake, 4, 5, fake, fake, fake, 1 << 30, fake,
                                     None) == ptq.ERR_INVALID_ARG                                   # unknown mode
    assert lib.ptq_quantize_layer(fake, 4, 8, 8, fake, None, fake, fake, 4, fake, None, None, None, fake, 1 << 30,
                                  fake, None) == ptq.ERR_INVALID_ARG
    assert lib.ptq_quantize_layer(fake, 4, 8, 8, fake, fake, fake, fake, 1, fake, None, None, None, fake, 1 << 30,
                                  fake, None) == ptq.ERR_INVALID_ARG                                # bits < 2
    assert lib.ptq_quantize_layer(fake, 4, 8, 8, fake, fake, fake, fake, 4, fake, None, None, None, fake, 64,
                                  fake, None) == ptq.ERR_WORKSPACE


def test_new_entry_points_check_their_arguments_on_the_host(lib):
    from paper_2509_05576_b200 import ptq
    vp = ctypes.c_void_p
    fake = vp(4096)
    assert lib.ptq_sort_scores(None, 8, 0, fake, None) == ptq.ERR_INVALID_ARG
    assert lib.ptq_sort_scores(fake, 0, 0, fake, None) == ptq.ERR_INVALID_ARG
    assert lib.ptq_selftest_wait_timeout(2, 1000, fake, 64, fake, None) == ptq.ERR_INVALID_ARG
    assert lib.ptq_selftest_wait_timeout(0, 0, fake, 64, fake, None) == ptq.ERR_INVALID_ARG
    assert lib.ptq_selftest_wait_timeout(0, 10 ** 12, fake, 64, fake, None) == ptq.ERR_INVALID_ARG   # beyond the library's own limit
    assert lib.ptq_selftest_wait_timeout(0, 1000, fake, 8, fake, None) == ptq.ERR_WORKSPACE
    flops = ctypes.c_double(0.0)
    assert lib.ptq_fp64_probe(2, 10, fake, ctypes.byref(flops), None) == ptq.ERR_INVALID_ARG
    assert lib.ptq_fp64_probe(0, 0, fake, ctypes.byref(flops), None) == ptq.ERR_INVALID_ARG
    # score modes: a direction flag on a valid mode is accepted by the argument check, anything else is not
    args = (fake, 4, 4, 4, fake, fake, fake, 4)
    assert lib.ptq_sensitivity_order(*args, 5, fake, fake, fake, 1 << 20, fake, None) == ptq.ERR_INVALID_ARG
    assert lib.ptq_sensitivity_order(*args, 32, fake, fake, fake, 1 << 20, fake, None) == ptq.ERR_INVALID_ARG
    assert lib.ptq_sensitivity_order(*args, ptq.SCORE_W | ptq.SCORE_ASCENDING, fake, fake, None, 0, fake, None) == ptq.ERR_WORKSPACE
    # dynamic re-ranking: rounds end on the 64-column block grid
    dyn = (fake, 8, 200, 200, fake, fake, fake, 4, 0)
    assert lib.ptq_quantize_layer_dynamic(*dyn, 100, fake, None, fake, None, None, fake, 1 << 40, fake, None) == ptq.ERR_UNSUPPORTED
    assert lib.ptq_quantize_layer_dynamic(*dyn, 0, fake, None, fake, None, None, fake, 1 << 40, fake, None) == ptq.ERR_INVALID_ARG
    assert lib.ptq_quantize_layer_dynamic(*dyn, 64, fake, None, fake, None, None, fake, 64, fake, None) == ptq.ERR_WORKSPACE
    # sizes beyond what the launch grid can index are refused, not launched
    assert lib.ptq_quantize_layer(fake, 70000, 8, 8, fake, fake, fake, fake, 4, fake, None, None, None, fake, 1 << 40,
                                  fake, None) == ptq.ERR_UNSUPPORTED


def test_binding_refuses_cpu_tensors(lib):
    import torch
    from paper_2509_05576_b200 import ptq
    with pytest.raises(ValueError):
        ptq.hessian_accumulate(torch.zeros(4, 4, dtype=torch.float64), torch.zeros(4, 8), None, None)


def test_layer_shape_sets_have_the_published_weight_counts():
    """The synthetic layer sets take nothing but shapes from the networks of Sec. 6: their weight totals are the
    well-known convolution + classifier weight counts of those architectures."""
    from paper_2509_05576_b200 import workloads as wl
    assert sum(r * c for _, r, c in wl.resnet50_shapes()) == 25_502_912 and len(wl.resnet50_shapes()) == 54
    assert sum(r * c for _, r, c in wl.resnet_basic_shapes((2, 2, 2, 2))) == 11_678_912      # ResNet-18
    assert sum(r * c for _, r, c in wl.resnet_basic_shapes((3, 4, 6, 3))) == 21_779_648      # ResNet-34
    assert sum(r * c for _, r, c in wl.yolov5s_shapes()[:-1]) == 7_215_616
    for spec in wl.conv_cases() + wl.resnet_conv_specs():
        oh, ow = spec.out_hw
        assert oh >= 1 and ow >= 1 and spec.n == spec.batch * oh * ow and spec.cols == spec.channels * spec.kh * spec.kw
    # the convolution whose unfolded input is the benchmark layer's shape
    c = wl.resnet_conv_specs()[0]
    assert (c.out_channels, c.cols) == (256, 2304) and abs(c.n - 4096) < 64


def test_conv_entry_point_rejects_bad_arguments_without_a_gpu(lib):
    from paper_2509_05576_b200 import ptq
    fake = ctypes.c_void_p(4096)
    f = lib.ptq_hessian_accumulate_conv
    assert f(fake, fake, 1, 3, 8, 8, 3, 3, 0, 1, fake, 1 << 30, fake, None) == ptq.ERR_INVALID_ARG      # stride 0
    assert f(fake, fake, 1, 3, 8, 8, 12, 3, 1, 1, fake, 1 << 30, fake, None) == ptq.ERR_INVALID_ARG     # kernel > image
    assert f(None, fake, 1, 3, 8, 8, 3, 3, 1, 1, fake, 1 << 30, fake, None) == ptq.ERR_INVALID_ARG
    assert f(fake, fake, 1, 3, 8, 8, 3, 3, 1, 1, fake, 16, fake, None) == ptq.ERR_WORKSPACE
    assert f(fake, fake, 1, 1 << 18, 8, 8, 3, 3, 1, 1, fake, 1 << 40, fake, None) == ptq.ERR_UNSUPPORTED   # cols > 2^20


def test_layer_set_plan_deals_every_layer_once_and_balances_the_streams():
    """Host logic of ptq.LayerSet: the plan is a permutation of the layers, the longest layers are issued first, no
    stream's estimated load exceeds the mean by more than the longest layer, and round-robin is kept when asked for."""
    from paper_2509_05576_b200 import ptq
    from paper_2509_05576_b200 import workloads as wl
    shapes = [(s.rows, s.cols) for s in wl.config3()]
    for n_streams in (1, 3, 8):
        plan = ptq.plan_layer_set(shapes, n_streams)
        assert sorted(i for i, _ in plan) == list(range(len(shapes)))
        assert all(0 <= k < n_streams for _, k in plan)
        est = [ptq.estimate_layer_ms(r, c) for r, c in shapes]
        issued = [est[i] for i, _ in plan]
        assert issued == sorted(issued, reverse=True)
        load = [0.0] * n_streams
        for i, k in plan:
            load[k] += est[i]
        assert max(load) <= sum(est) / n_streams + max(est) + 1e-9
    assert ptq.plan_layer_set(shapes[:5], 2, longest_first=False) == [(0, 0), (1, 1), (2, 0), (3, 1), (4, 0)]
    # wider and taller layers are estimated longer
    assert ptq.estimate_layer_ms(512, 4608) > ptq.estimate_layer_ms(256, 2304) > ptq.estimate_layer_ms(64, 64)
    assert ptq.estimate_layer_ms(4096, 4096) > ptq.estimate_layer_ms(512, 4096)
