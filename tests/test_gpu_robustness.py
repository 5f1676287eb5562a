"""Failure detection and checkpoint/resume on the GPU, without faulting, trapping or hanging anything:
bounded waits report through a status word, non-finite inputs are latched, state round-trips bit-exactly."""
import numpy as np
import pytest

from parity_util import Case, make_inputs, make_plan, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch():
    import torch
    return torch


def _tensors(case, inp, torch):
    n = len(case.shapes)
    G = [to_dev(inp["G"][i], case.dtype, torch, "cuda:0") for i in range(n)]
    A = [to_dev(inp["anchors"][i][0], case.dtype, torch, "cuda:0") for i in range(n)]
    W = [torch.from_numpy(inp["W"][i].copy()).cuda() for i in range(n)]
    m = [torch.from_numpy(inp["m"][i].copy()).cuda() for i in range(n)]
    v = [torch.from_numpy(inp["v"][i].copy()).cuda() for i in range(n)]
    return G, A, W, m, v


def test_bounded_wait_reports_timeout_and_context_stays_usable(torch):
    case = Case(shapes=[(256, 384)], rank=16, tokens=128)
    inp = make_inputs(case)
    plan = make_plan(case, torch)
    assert plan.get_device_status() == 0
    plan.debug_wait_probe(2048)                      # a wait nothing will satisfy; gives up after 2048 polls
    assert plan.get_device_status() == -9            # SC_ERR_TIMEOUT, latched ...
    assert plan.get_device_status() == 0             # ... and cleared by the read
    # the plan and the CUDA context are still fine
    G, A, W, m, v = _tensors(case, inp, torch)
    plan.anchor_update(A, 0)
    assert plan.correct_and_step(G, W, m, v, 100) == 0
    torch.cuda.synchronize()
    assert plan.get_device_status() == 0 and bool(torch.isfinite(W[0]).all())


@pytest.mark.parametrize("engine", [0, 1])
def test_non_finite_gradient_is_latched(torch, engine):
    case = Case(shapes=[(256, 384), (256, 384)], rank=16, tokens=128, engine=engine)
    inp = make_inputs(case)
    plan = make_plan(case, torch)
    G, A, W, m, v = _tensors(case, inp, torch)
    plan.anchor_update(A, 0)
    G[1][17, 33] = float("nan")
    plan.correct_and_step(G, W, m, v, 100)
    assert plan.get_device_status() == -10           # SC_ERR_NONFINITE
    assert plan.get_device_status() == 0


@pytest.mark.parametrize("engine", [0, 1])
def test_state_export_import_continues_bit_identically(torch, engine):
    import paper_2609_14339_b200 as sc
    case = Case(shapes=[(256, 384), (200, 136), (256, 384)], rank=12, tokens=128, planted=4, tau_p=30.0, engine=engine,
                dtype="bf16")
    inp = make_inputs(case)
    a = make_plan(case, torch)
    G, A, W, m, v = _tensors(case, inp, torch)
    a.anchor_update([A[0], None, A[2]], 7)           # one matrix has no basis yet
    blob = a.state_export()
    b = make_plan(case, torch)
    b.state_import(blob)
    assert b.get_anchor_info() == (7, 2)
    W2, m2, v2 = [x.clone() for x in W], [x.clone() for x in m], [x.clone() for x in v]
    a.correct_and_step(G, W, m, v, 100)
    b.correct_and_step(G, W2, m2, v2, 100)
    torch.cuda.synchronize()
    for x, y in zip(W + m + v, W2 + m2 + v2):
        assert torch.equal(x, y)
    # a blob from a plan of another rank is refused
    other = make_plan(Case(**{**case.__dict__, "rank": 8}), torch)
    with pytest.raises(sc.SCError) as e:
        other.state_import(blob)
    assert e.value.status in (-2, -5)
    # the same shapes in another order (equal totals, equal rank) are refused too: SC_ERR_SHAPE
    perm = make_plan(Case(**{**case.__dict__, "shapes": [case.shapes[1], case.shapes[0], case.shapes[2]]}), torch)
    with pytest.raises(sc.SCError) as e:
        perm.state_import(blob)
    assert e.value.status == -2
    # a plan with another tau_p gets its own filter weights from the imported singular values (Eq. 2), not the blob's
    c2 = make_plan(Case(**{**case.__dict__, "tau_p": 5.0}), torch)
    c2.state_import(blob)
    _, s0, _ = c2.export_basis(0)
    gp = [torch.zeros(sh, dtype=torch.float32, device="cuda:0") for sh in case.shapes]
    c2.set_debug_gproj_out(gp)
    W3, m3, v3 = [x.clone() for x in W2], [x.clone() for x in m2], [x.clone() for x in v2]
    c2.correct_and_step(G, W3, m3, v3, 101)
    fresh = make_plan(Case(**{**case.__dict__, "tau_p": 5.0}), torch)
    fresh.anchor_update([A[0], None, A[2]], 7)
    gq = [torch.zeros(sh, dtype=torch.float32, device="cuda:0") for sh in case.shapes]
    fresh.set_debug_gproj_out(gq)
    W4, m4, v4 = [x.clone() for x in W2], [x.clone() for x in m2], [x.clone() for x in v2]
    fresh.correct_and_step(G, W4, m4, v4, 101)
    torch.cuda.synchronize()
    assert all(torch.equal(x, y) for x, y in zip(gp, gq))


def test_two_latched_conditions_are_reported_one_after_the_other(torch):
    case = Case(shapes=[(256, 384)], rank=16, tokens=128)
    inp = make_inputs(case)
    plan = make_plan(case, torch)
    G, A, W, m, v = _tensors(case, inp, torch)
    plan.anchor_update(A, 0)
    G[0][3, 5] = float("inf")
    plan.correct_and_step(G, W, m, v, 100)           # latches the non-finite bit
    plan.debug_wait_probe(1024)                      # latches the time-out bit as well
    assert plan.get_device_status() == -9
    assert plan.get_device_status() == -10
    assert plan.get_device_status() == 0
