"""Parity of EVERY layer of the ResNet-50-shaped and YOLOv5s-shaped sets and of the scaling shapes against the CPU
oracle, layer by layer, at full size (a few minutes, nearly all of it oracle time on the host)."""
import numpy as np
import pytest

from paper_2509_05576_b200 import workloads as wl
from test_gpu_configs import _full, _row_subset_parity

pytestmark = pytest.mark.gpu

_SETS = {"c3": wl.config3(), "c4w8": wl.config4(bits=(8,)), "c4w4": wl.config4(bits=(4,))}


def _ids(specs):
    return [s.name for s in specs]


@pytest.mark.parametrize("spec", _SETS["c3"], ids=_ids(_SETS["c3"]))
def test_resnet50_set(spec):
    if spec.cols > 2304:
        assert _row_subset_parity(spec, 32, seed=spec.seed) == 0
    else:
        nm, _, _ = _full(spec)
        assert nm == 0


@pytest.mark.parametrize("spec", _SETS["c4w8"] + _SETS["c4w4"], ids=_ids(_SETS["c4w8"] + _SETS["c4w4"]))
def test_yolov5s_set(spec):
    if spec.cols > 2304:
        assert _row_subset_parity(spec, 32, seed=spec.seed) == 0
    else:
        nm, _, _ = _full(spec)
        assert nm == 0


_C5 = [s for s in wl.config5() if s.cols <= 4608]


@pytest.mark.parametrize("spec", _C5, ids=_ids(_C5))
def test_scaling_shapes(spec):
    """1024x1024 in full; 2048x4608 and 4096x4096 with the oracle sweep on 32 seeded rows.  (4096x11008 is beyond the
    oracle's reach: its Eq. 12 loop alone is 4.4e11 multiply-adds per pass over a 970 MB matrix.)"""
    if spec.cols > 1024:
        assert _row_subset_parity(spec, 32, seed=spec.seed) == 0
    else:
        nm, _, _ = _full(spec)
        assert nm == 0
