"""sc_project_static: the projection X = U^T G V for callers that cannot allocate device memory.

Some users reach this library from a place where neither cudaMalloc nor a workspace is available (the
framework's caching allocator already owns HBM, or the path must not synchronise the device). The entry point
keeps its intermediates in a fixed array inside the library. This test calls it through the C ABI twice in a
row - a large matrix first, a smaller one second, so the second call runs on top of the first call's leftovers -
and checks both results against the projection the plan-based entry points compute, within the tolerance the
other projection tests use for X (5e-4 relative Frobenius: the plan path forms X on tf32 tensor cores), and against
the fp64 oracle's X = U^T G V on the same device arrays at 1e-5 (this entry point works in plain fp32 FMA).

Collected last on purpose (file name): a run that stops at the first failure has then run everything else.
"""
import ctypes as C

import numpy as np
import pytest

from oracle import spectral_oracle as so
from parity_util import Case, GpuRun, make_inputs, rel

pytestmark = pytest.mark.gpu
TOL = 5e-4
TOL_ORACLE = 1e-5


@pytest.fixture(scope="module")
def torch():
    import torch
    return torch


def _plan_projection(case, torch):
    """U, V, G on the device and X from the existing entry points (sc_correct_and_step + sc_export_projection)."""
    from parity_util import to_dev
    inp = make_inputs(case)
    g = GpuRun(case, inp, torch)
    out = []
    for i in range(len(case.shapes)):
        U, s, V = g.plan.export_basis(i)
        T, X = g.plan.export_projection(i)
        G = to_dev(inp["G"][i], case.dtype, torch, "cuda:0")
        out.append((G, U.contiguous(), V.contiguous(), X.double().cpu().numpy()))
    torch.cuda.synchronize()
    return g, out


def test_two_calls_in_a_row_match_the_plan_path(torch):
    import paper_2609_14339_b200 as sc
    big = Case(shapes=[(512, 1024)], rank=64, tokens=512, keep=0.1, planted=32, seed=2, tau_p=100.0)
    small = Case(shapes=[(330, 264)], rank=5, tokens=192, keep=0.5, planted=3, seed=3, tau_p=40.0, dtype="fp32", engine=1)
    gb, (b,) = _plan_projection(big, torch)
    gs, (s,) = _plan_projection(small, torch)
    Xb = torch.empty((64, 64), dtype=torch.float32, device="cuda:0")
    Xs = torch.empty((5, 5), dtype=torch.float32, device="cuda:0")
    sc.project_static(b[0], b[1], b[2], X_out=Xb)        # first call: bf16 gradient, rank 64
    sc.project_static(s[0], s[1], s[2], X_out=Xs)        # second call, same stream, on the first call's leftovers
    torch.cuda.synchronize()
    assert rel(Xb.double().cpu().numpy(), b[3]) < TOL
    assert rel(Xs.double().cpu().numpy(), s[3]) < TOL
    for X, (G, U, V, _) in ((Xb, b), (Xs, s)):
        want = so.project(U.double().cpu().numpy(), G.double().cpu().numpy(), V.double().cpu().numpy())
        assert rel(X.double().cpu().numpy(), want) <= TOL_ORACLE
    # and once more in the opposite order, results unchanged
    Xs2 = sc.project_static(s[0], s[1], s[2])
    Xb2 = sc.project_static(b[0], b[1], b[2])
    torch.cuda.synchronize()
    assert torch.equal(Xs2, Xs) and torch.equal(Xb2, Xb)


def test_rejects_sizes_beyond_the_fixed_scratch(torch):
    import paper_2609_14339_b200 as sc
    lib = sc.load_library()
    x = torch.zeros(16, device="cuda:0")
    p = x.data_ptr()
    # 40000 x 64 floats of T alone exceed the 2,097,152-float array
    assert lib.sc_project_static(p, 0, p, p, 40000, 4096, 64, p, None) == -11
    assert lib.sc_project_static(p, 0, p, p, 128, 128, 300, p, None) == -2        # rank > rows
    assert lib.sc_project_static(None, 0, p, p, 128, 128, 8, p, None) == -1
    assert lib.sc_project_static(p, 5, p, p, 128, 128, 8, p, None) == -3
    torch.cuda.synchronize()
