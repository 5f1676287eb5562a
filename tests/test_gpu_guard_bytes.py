"""Out-of-bounds evidence without a memory checker: every buffer the library is given (gradients, weights, AdamW
moments, the bf16 weight copy, the debug G_proj output, the workspace, mask and weight-gradient operands) sits inside a
larger allocation filled with a poison byte, and after the calls every guard byte must still hold it.  Ragged shapes
(smaller than a tile, one row or column past a tile edge) on both engines: the TMA stores there are clipped by the
tensor maps, the CUDA-core kernels by their bounds checks.  Nothing here is expected to fault."""
import numpy as np
import pytest

from parity_util import Case, make_inputs

pytestmark = pytest.mark.gpu
POISON = 0xA5
GUARD = 8192          # bytes on either side


@pytest.fixture(scope="module")
def torch():
    import torch
    return torch


class Guarded:
    """A typed CUDA tensor carved out of the middle of a poison-filled allocation."""

    def __init__(self, torch, shape, dtype, src=None, align=256):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.raw = torch.full((n + 2 * GUARD + align,), POISON, dtype=torch.uint8, device="cuda:0")
        self.off = GUARD + (-(self.raw.data_ptr() + GUARD)) % align
        self.n = n
        self.t = self.raw[self.off:self.off + n].view(dtype).view(shape)
        if src is not None:
            self.t.copy_(src)
        self.torch = torch

    def intact(self):
        lo, hi = self.raw[:self.off], self.raw[self.off + self.n:]
        return bool((lo == POISON).all()) and bool((hi == POISON).all())


def _bf16(torch, bits):
    return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16)


@pytest.mark.parametrize("engine", [0, 1])
def test_anchor_update_and_step_leave_every_guard_byte_intact(torch, engine):
    import paper_2609_14339_b200 as sc
    shapes = [(200, 136), (72, 520), (16, 64), (129, 200), (200, 136)]
    case = Case(shapes=shapes, rank=5, tokens=96, keep=0.5, planted=2, tau_p=20.0, engine=engine, max_grad_norm=0.5)
    inp = make_inputs(case)
    hp = sc.Hparams.default(tau_p=case.tau_p, lr=case.lr, weight_decay=case.weight_decay, engine=engine, collect_stats=1,
                            max_grad_norm=case.max_grad_norm, warm_start=1)
    ws = Guarded(torch, (sc.Plan.workspace_bytes_for(shapes, case.rank, hp),), torch.uint8)
    plan = sc.Plan(shapes, case.rank, case.keep, hp, workspace=ws.t)
    assert plan.uses_tensor_cores() == (engine == 0)
    f32, b16 = torch.float32, torch.bfloat16
    G = [Guarded(torch, s, b16, _bf16(torch, inp["G"][i])) for i, s in enumerate(shapes)]
    A = [Guarded(torch, s, b16, _bf16(torch, inp["anchors"][i][0])) for i, s in enumerate(shapes)]
    W = [Guarded(torch, s, f32, torch.from_numpy(inp["W"][i])) for i, s in enumerate(shapes)]
    m = [Guarded(torch, s, f32, torch.from_numpy(inp["m"][i])) for i, s in enumerate(shapes)]
    v = [Guarded(torch, s, f32, torch.from_numpy(inp["v"][i])) for i, s in enumerate(shapes)]
    Wb = [Guarded(torch, s, b16) for s in shapes]
    gp = [Guarded(torch, s, f32) for s in shapes]
    plan.set_debug_gproj_out([x.t for x in gp])
    t = lambda xs: [x.t for x in xs]
    for step in range(3):                                   # cold arrival, warm arrival, partial arrival
        anc = t(A) if step < 2 else [A[0].t, None, A[2].t, None, None]
        plan.anchor_update(anc, step)
        assert plan.correct_and_step(t(G), t(W), t(m), t(v), 100 + step, params_bf16=t(Wb)) == 0
    torch.cuda.synchronize()
    assert plan.get_device_status() == 0
    U, s_, V = plan.export_basis(3)
    for name, group in (("workspace", [ws]), ("G", G), ("G_anc", A), ("W", W), ("m", m), ("v", v), ("Wb", Wb), ("gproj", gp)):
        for i, x in enumerate(group):
            assert x.intact(), (name, i)
    # the calls did real work: state moved, the bf16 copy follows the weights, inputs are untouched
    for i in range(len(shapes)):
        assert not torch.equal(W[i].t.cpu(), torch.from_numpy(inp["W"][i]))
        assert torch.equal(G[i].t.cpu(), _bf16(torch, inp["G"][i]))
        assert float((Wb[i].t.float() - W[i].t).abs().max()) < 1e-2
        assert bool(torch.isfinite(gp[i].t).all())
    plan.close()


def test_mask_and_weight_gradient_entry_points_leave_guards_intact(torch):
    import paper_2609_14339_b200 as sc
    rng = np.random.default_rng(7)
    for tokens, rows, cols in ((100, 72, 136), (257, 264, 520), (64, 8, 8)):
        X = Guarded(torch, (tokens, cols), torch.bfloat16, torch.from_numpy(rng.standard_normal((tokens, cols)).astype(np.float32)))
        dY = Guarded(torch, (tokens, rows), torch.bfloat16, torch.from_numpy(rng.standard_normal((tokens, rows)).astype(np.float32)))
        Xm = Guarded(torch, (tokens, cols), torch.bfloat16)
        for odt in (torch.bfloat16, torch.float32):
            Gout = Guarded(torch, (rows, cols), odt)
            status = Guarded(torch, (1,), torch.int32, torch.zeros(1, dtype=torch.int32))
            sc.masked_weight_grad(dY.t, X.t, 0.25, seed=3, layer=1, step=2, Xm=Xm.t, out=Gout.t, status=status.t)
            torch.cuda.synchronize()
            assert int(status.t.item()) == 0
            assert all(x.intact() for x in (X, dY, Xm, Gout, status)), (tokens, rows, cols, odt)
            assert float(Gout.t.float().abs().max()) > 0
    for tokens, feats in ((33, 37), (9, 5), (64, 4096)):
        X = Guarded(torch, (tokens, feats), torch.bfloat16, torch.from_numpy(rng.standard_normal((tokens, feats)).astype(np.float32)), align=16)
        out = Guarded(torch, (tokens, feats), torch.bfloat16, align=16)
        sc.apply_prf_mask(X.t, 0.3, seed=1, layer=0, step=5, rescale=True, out=out.t, exact_k=True)
        torch.cuda.synchronize()
        assert X.intact() and out.intact(), (tokens, feats)
    X = Guarded(torch, (40, 72), torch.bfloat16, torch.from_numpy(rng.standard_normal((40, 72)).astype(np.float32)))
    out = Guarded(torch, (40, 72), torch.bfloat16)
    sc.apply_prf_mask(X.t, 0.3, seed=1, layer=0, step=5, out=out.t)
    torch.cuda.synchronize()
    assert X.intact() and out.intact()
