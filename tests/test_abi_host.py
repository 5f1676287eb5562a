"""Host-side checks that need no GPU: the library loads, exports every declared symbol, and the
host-only entry points (defaults, workspace sizing, status strings, argument checks) behave."""
import ctypes as C
import os
import re

import pytest

import paper_2609_14339_b200 as sc
from paper_2609_14339_b200 import binding as b

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_14339_b200 import build
    build.build()
    return b.load_library()


def test_library_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "spectral_correction.h")).read()
    declared = set(re.findall(r"SC_API\s+[\w\s\*]+?\b(sc_\w+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(b.EXPORTS), (declared ^ set(b.EXPORTS))
    for name in declared:
        assert getattr(lib, name) is not None


def test_defaults_follow_the_paper(lib):
    hp = sc.Hparams.default()
    assert abs(hp.alpha - 0.3) < 1e-7 and abs(hp.tau_p - 1e-3) < 1e-9          # ablation-table defaults
    assert abs(hp.lr - 2e-5) < 1e-11 and abs(hp.beta1 - 0.9) < 1e-7 and abs(hp.beta2 - 0.999) < 1e-7
    assert hp.max_grad_norm == 0.0 and hp.grads_prescaled == 1 and hp.grad_dtype == sc.SC_DTYPE_BF16


def _ws(lib, shapes, rank, hp):
    arr = (b.Shape * len(shapes))(*[b.Shape(m, n) for m, n in shapes])
    return lib.sc_plan_workspace_bytes(arr, len(shapes), rank, C.byref(hp))


def test_workspace_sizing(lib):
    hp = sc.Hparams.default()
    one = _ws(lib, [(512, 256)], 16, hp)
    assert one >= 512 * 256 * 4                              # holds at least the anchor momentum
    two = _ws(lib, [(512, 256)] * 2, 16, hp)
    assert two > one and two < 2 * one + (1 << 20)
    assert _ws(lib, [(512, 256)], 32, hp) > one              # grows with rank
    # the 8B-shaped set fits comfortably next to params and optimizer state in 180 GB
    from synth.generator import config_shapes
    big = _ws(lib, config_shapes("llama8b"), 64, hp)
    assert 26e9 < big < 40e9


def test_workspace_rejects_bad_input(lib):
    hp = sc.Hparams.default()
    assert _ws(lib, [(8, 8)], 9, hp) == 0                    # rank > min(m, n)
    assert _ws(lib, [(0, 8)], 1, hp) == 0
    assert _ws(lib, [(512, 512)], 300, hp) == 0              # rank > 256
    hp2 = sc.Hparams.default(sketch_width=4)
    assert _ws(lib, [(64, 64)], 8, hp2) == 0                 # l < rank
    hp3 = sc.Hparams.default(alpha=1.5)
    assert _ws(lib, [(64, 64)], 8, hp3) == 0


def test_status_strings(lib):
    seen = set()
    for code in list(range(-11, 2)):
        s = sc.status_string(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 13
    assert sc.status_string(77) == "unknown status"


def test_create_rejects_bad_arguments_before_touching_cuda(lib):
    hp = sc.Hparams.default()
    arr = (b.Shape * 1)(b.Shape(64, 64))
    h = C.c_void_p()
    assert lib.sc_plan_create(C.byref(h), arr, 1, 8, C.c_float(0.0), C.byref(hp), 256, 1 << 20, None) == -1  # keep = 0
    assert lib.sc_plan_create(C.byref(h), arr, 1, 8, C.c_float(0.5), C.byref(hp), None, 1 << 20, None) == -1  # no workspace
    assert lib.sc_plan_create(C.byref(h), arr, 1, 8, C.c_float(0.5), C.byref(hp), 264, 1 << 20, None) == -4  # misaligned
    assert lib.sc_plan_create(C.byref(h), arr, 1, 80, C.c_float(0.5), C.byref(hp), 256, 1 << 20, None) == -2  # rank > n
    hp.grad_dtype = 7
    assert lib.sc_plan_create(C.byref(h), arr, 1, 8, C.c_float(0.5), C.byref(hp), 256, 1 << 20, None) == -3
    assert lib.sc_plan_destroy(None) == -1
    assert lib.sc_anchor_update(None, None, 0) == -1
