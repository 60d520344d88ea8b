"""GPU parity on the named workloads at their full layer sizes.  Every output
element of the VGG-16 stack is compared; for the batched ResNet stacks and the
sweep the whole batch runs on the GPU in the benchmark's launch configuration
and sampled images (first and last of the batch) are compared element by
element -- images are independent, so the oracle computes them one by one."""
import numpy as np
import pytest

from paper_2206_10620_b200 import workloads as wl
from _gpu_util import compare, pack, run_gpu

pytestmark = pytest.mark.gpu


def test_vgg16_every_layer_every_element():
    for spec in wl.config_vgg16():
        d = wl.make_layer(spec)
        compare(d, run_gpu(pack(d), d.x, d.bias, True))


def _sampled_batch(spec, images):
    d = wl.make_layer(spec)
    y = run_gpu(pack(d), d.x, d.bias, True)
    for i in images:
        compare(d, y[i:i + 1], x=d.x[i:i + 1])


def test_resnet50_layers_sampled_images():
    seen = set()
    for spec in wl.config_resnet50():
        key = (spec.c_in, spec.h, spec.stride)
        if key in seen:
            continue                                  # one layer per distinct shape
        seen.add(key)
        _sampled_batch(spec, [0, spec.n - 1])


def test_resnet18_layers_sampled_images():
    seen = set()
    for spec in wl.config_resnet18():
        key = (spec.c_in, spec.c_out, spec.h, spec.stride)
        if key in seen:
            continue
        seen.add(key)
        _sampled_batch(spec, [0, spec.n - 1])


def test_sweep_points():
    pts = [s for s in wl.config_sweep() if s.n in (1, 64)]
    for spec in pts[::3]:
        _sampled_batch(spec, [0] if spec.n == 1 else [0, spec.n - 1])
