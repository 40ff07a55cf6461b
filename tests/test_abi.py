"""The C-ABI library loads, exports every function include/harp.h declares, and
rejects bad input before touching CUDA (runs without a GPU)."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2605_29843_b200 as harp
from paper_2605_29843_b200 import build as harp_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    harp_build.build()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "harp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(harp_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    names = declared_functions()
    assert {"harp_plan_create", "harp_apply", "harp_apply_two_sided", "harp_plan_destroy"} <= set(names)
    L = harp.lib()
    for n in names:
        assert getattr(L, n) is not None, n


def test_binding_has_the_same_names():
    for n in declared_functions():
        if n in ("harp_plan_destroy", "harp_status_string", "harp_apply_ex"):
            continue                     # owned by Plan.__del__ / status_string / harp_apply(kernel=)
        assert hasattr(harp, n), n


def _eye_blocks(d, radices):
    return [np.broadcast_to(np.eye(b, dtype=np.float32), (d // b, b, b)).copy() for b in radices]


@pytest.mark.parametrize("kwargs,code", [
    (dict(d=8, radices=(2, 2, 3)), 3),                 # product != d
    (dict(d=8, radices=(2, 4, 1)), 3),                 # radix < 2
    (dict(d=1, radices=(1,)), 2),                      # d < 2
    (dict(d=8, radices=(2, 2, 2), perm=[0, 1, 2, 3, 4, 5, 6, 6]), 4),
    (dict(d=8, radices=(2, 2, 2), perm=[0, 1, 2, 3, 4, 5, 6, 8]), 4),
    (dict(d=8, radices=(2, 2, 2), signs=[1, 1, 1, 0, 1, 1, 1, 1]), 5),
])
def test_plan_validation_codes(kwargs, code):
    d, radices = kwargs["d"], kwargs["radices"]
    blocks = [np.zeros((max(1, d // max(b, 1)), max(b, 1), max(b, 1)), np.float32) for b in radices]
    st, plan = harp.harp_plan_create_status(d, radices, kwargs.get("perm"), kwargs.get("signs"), blocks)
    assert st == code and plan is None
    assert isinstance(harp.status_string(st), str) and harp.status_string(st) != "ok"


def test_null_arguments():
    L = harp.lib()
    assert L.harp_apply(None, None, 4, 0, 0, None) == 1
    assert L.harp_apply_two_sided(None, 0, None, None, None, None) == 1
    assert L.harp_plan_dim(None) == -1
    assert L.harp_two_sided_scratch_bytes(None, None, 0) == 0
    out = ctypes.c_void_p()
    assert L.harp_plan_create(ctypes.byref(out), 8, 3, None, None, None, None) == 1
    L.harp_plan_destroy(None)
    assert harp.status_string(0) == "ok"
    assert harp.harp_launch_count() >= 0


def test_null_arguments_of_the_widened_entry_points():
    """Passes, gradient and diagnostics reject bad arguments before any CUDA call."""
    L = harp.lib()
    assert L.harp_apply_passes(None, 1, None, 4, 0, 0, None) == 1
    arr = (ctypes.c_void_p * 1)(None)
    assert L.harp_apply_passes(arr, 1, None, 4, 0, 0, None) == 1          # a NULL plan in the list
    assert L.harp_apply_passes(arr, 0, None, 4, 0, 0, None) == 3          # no passes
    assert L.harp_grad_blocks(None, None, None, 4, 0, None, 0, None) == 1
    assert L.harp_plan_n_params(None) == -1
    buf = (ctypes.c_double * 4)()
    assert L.harp_weight_incoherence(None, 4, 4, 0, buf, None) == 1
    assert L.harp_weight_incoherence(buf, 0, 4, 0, buf, None) == 2        # empty matrix
    assert L.harp_weight_incoherence(buf, 4, 4, 7, buf, None) == 6        # unknown dtype
    assert L.harp_offblock_energy(None, 4, 2, 0, buf, None) == 1
    assert L.harp_offblock_energy(buf, 4, 5, 0, buf, None) == 2           # block larger than n
    assert L.harp_offblock_energy(buf, 4, 0, 0, buf, None) == 2
    assert L.harp_diag_weighted_error(None, buf, 2, 2, 0, buf, 0, buf, None) == 1


def test_no_gpu_means_an_error_not_a_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    st, plan = harp.harp_plan_create_status(8, (2, 2, 2), None, None, _eye_blocks(8, (2, 2, 2)))
    assert st in (9, 10) and plan is None
