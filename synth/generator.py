"""Seeded synthetic inputs for the spectral-correction step.

This module only produces *input arrays* (activations, output gradients, column
keep masks, and the weight gradients formed from them).  It holds none of the
method's arithmetic: no EMA, no SVD, no filter, no optimizer.  Both the CPU
oracle tests and the GPU tests feed the arrays produced here to their side.

Recipe (per weight matrix W in R^{m x n}, per step, T tokens):

    X  = Z_x + a * C * P_x^T          (T x n)   activations
    dY = Z_y + a * C * P_y^T          (T x m)   output gradients
    Z_x, Z_y, C ~ iid N(0, 1), C in R^{T x k} fresh per batch,
    P_x (n x k), P_y (m x k): fixed orthonormal per matrix (the planted shared component),
    a^4 = SNR * m * n / (T * k)       so planted and noise parts of dY^T X have equal energy at SNR 1,
    Mk ~ Bernoulli(keep) iid on T x n (column-keep mask over activations),
    G_mask = dY^T (X * Mk) / keep,    G_anc = dY'^T X' from an independent unmasked batch.

Random activation masking with receiver-side rescaling is the scheme analysed in
the paper's "random vs top-K" appendix (Bernoulli(1-p) independent across
(token, feature), rescaled by 1/(1-p)); keep = 1 - p.

Streams are keyed on (seed, layer, matrix id, step, tensor id) so any array can
be regenerated on its own.  Two backends: NumPy (Philox) for CPU-sized cases and
torch (device generator) for cases that only fit on the GPU.  The two backends
do not produce the same numbers; a test always uses one backend for both sides.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

TENSOR_X, TENSOR_DY, TENSOR_C, TENSOR_MASK, TENSOR_PX, TENSOR_PY, TENSOR_W, TENSOR_M, TENSOR_V = range(9)


@dataclass(frozen=True)
class GradSpec:
    m: int                 # out features (rows of W)
    n: int                 # in features (cols of W)
    tokens: int            # T
    keep: float = 1.0      # keep ratio = 1 - p_mask
    planted_rank: int = 0  # k
    snr: float = 1.0
    seed: int = 0
    layer: int = 0
    mat_id: int = 0


def _key(spec: GradSpec, step: int, tensor: int):
    return [int(spec.seed) & 0xFFFFFFFFFFFFFFFF,
            (int(spec.layer) << 40) ^ (int(spec.mat_id) << 28) ^ ((int(step) & 0xFFFFF) << 8) ^ int(tensor)]


def _rng(spec: GradSpec, step: int, tensor: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=_key(spec, step, tensor)))


def planted_amplitude(spec: GradSpec) -> float:
    if spec.planted_rank <= 0:
        return 0.0
    return float((spec.snr * spec.m * spec.n / (spec.tokens * spec.planted_rank)) ** 0.25)


def planted_directions(spec: GradSpec):
    """Fixed orthonormal P_x (n x k), P_y (m x k) for this matrix (independent of step)."""
    k = spec.planted_rank
    if k <= 0:
        return np.zeros((spec.n, 0)), np.zeros((spec.m, 0))
    Px, _ = np.linalg.qr(_rng(spec, 0, TENSOR_PX).standard_normal((spec.n, k)))
    Py, _ = np.linalg.qr(_rng(spec, 0, TENSOR_PY).standard_normal((spec.m, k)))
    return Px, Py


def batch(spec: GradSpec, step: int):
    """Activations X (T x n) and output gradients dY (T x m) of one batch, fp64."""
    X = _rng(spec, step, TENSOR_X).standard_normal((spec.tokens, spec.n))
    dY = _rng(spec, step, TENSOR_DY).standard_normal((spec.tokens, spec.m))
    if spec.planted_rank > 0:
        a = planted_amplitude(spec)
        C = _rng(spec, step, TENSOR_C).standard_normal((spec.tokens, spec.planted_rank))
        Px, Py = planted_directions(spec)
        X = X + a * (C @ Px.T)
        dY = dY + a * (C @ Py.T)
    return X, dY


def keep_mask(spec: GradSpec, step: int) -> np.ndarray:
    """Bernoulli(keep) mask over (token, input feature), as 0/1 fp64."""
    if spec.keep >= 1.0:
        return np.ones((spec.tokens, spec.n))
    u = _rng(spec, step, TENSOR_MASK).random((spec.tokens, spec.n))
    return (u < spec.keep).astype(np.float64)


def dense_gradient(spec: GradSpec, step: int) -> np.ndarray:
    """Unmasked weight gradient dY^T X (m x n), fp64 (not rounded)."""
    X, dY = batch(spec, step)
    return dY.T @ X


def masked_gradient(spec: GradSpec, step: int, rescale: bool = True) -> np.ndarray:
    """dY^T (X * Mk) / keep (m x n), fp64 (not rounded); rescale=False leaves out the 1/keep."""
    X, dY = batch(spec, step)
    G = dY.T @ (X * keep_mask(spec, step))
    return G / spec.keep if rescale else G


def anchor_gradient(spec: GradSpec, step: int) -> np.ndarray:
    """Unmasked gradient of an independent batch; callers pass step = t - staleness (offset into its own stream)."""
    return dense_gradient(spec, (1 << 19) + step)


def round_to(G: np.ndarray, dtype: str) -> np.ndarray:
    """Round once (RNE) to the gradient storage type; returns fp32 ndarray for 'fp32', uint16 bit patterns for 'bf16'."""
    if dtype == "fp32":
        return np.asarray(G, np.float32)
    if dtype == "bf16":
        return f32_to_bf16_bits(np.asarray(G, np.float32))
    raise ValueError(dtype)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    b = np.ascontiguousarray(x, np.float32).view(np.uint32)
    rounding = ((b >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    out = ((b + rounding) >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out = np.where(nan, np.uint16(0x7FC0), out)
    return out


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def stored_to_f64(arr: np.ndarray, dtype: str) -> np.ndarray:
    """The exact value of a stored gradient array, upcast to fp64."""
    return bf16_bits_to_f64(arr) if dtype == "bf16" else np.asarray(arr, np.float64)


def optimizer_state(spec: GradSpec, warmed: bool = True):
    """Seeded W, m, v (fp32 values).  warmed=True gives a state as after many steps (m ~ N, v > 0)."""
    W = (_rng(spec, 0, TENSOR_W).standard_normal((spec.m, spec.n)) * 0.02).astype(np.float32)
    if not warmed:
        return W, np.zeros_like(W), np.zeros_like(W)
    scale = float(np.sqrt(spec.tokens))
    m = (_rng(spec, 0, TENSOR_M).standard_normal((spec.m, spec.n)) * 0.3 * scale).astype(np.float32)
    v = ((_rng(spec, 0, TENSOR_V).random((spec.m, spec.n)) + 0.5) * scale * scale).astype(np.float32)
    return W, m, v


# ---------------------------------------------------------------------------
# Named parameter sets (shapes of the Llama-style layers the configs list)
# ---------------------------------------------------------------------------
def llama_layer_shapes(hidden: int, ffn: int, kv: int):
    """(m, n) of the seven linear weights of one decoder layer: q, k, v, o, gate, up, down."""
    return [(hidden, hidden), (kv, hidden), (kv, hidden), (hidden, hidden),
            (ffn, hidden), (ffn, hidden), (hidden, ffn)]


CONFIGS = {
    # name: layers, per-layer shapes, tokens, keep, planted rank k, rank r, grad dtype
    "c1_256": dict(layers=1, shapes=[(256, 256)], tokens=512, keep=0.25, k=0, r=8, dtype="fp32"),
    "llama1b": dict(layers=16, shapes=llama_layer_shapes(2048, 8192, 2048), tokens=2048, keep=0.1, k=16, r=32, dtype="bf16"),
    "llama8b": dict(layers=32, shapes=llama_layer_shapes(4096, 14336, 1024), tokens=4096, keep=0.1, k=32, r=64, dtype="bf16"),
    "ffn_sweep": dict(layers=1, shapes=[(14336, 4096)], tokens=4096, keep=0.1, k=32, r=64, dtype="bf16"),
    "llama70b_slice": dict(layers=8, shapes=llama_layer_shapes(8192, 28672, 1024), tokens=8192, keep=0.05, k=64, r=128, dtype="bf16"),
    # 24 of the 32 8B-shaped layers: the largest slice whose state still fits in 180 GB with a fourth fp32 array per weight
    "llama8b_24layers": dict(layers=24, shapes=llama_layer_shapes(4096, 14336, 1024), tokens=4096, keep=0.1, k=32, r=64, dtype="bf16"),
    # two 8B-shaped layers: small enough (6 GB resident) for multi-pass profiler captures of the short kernels
    "llama8b_2layers": dict(layers=2, shapes=llama_layer_shapes(4096, 14336, 1024), tokens=4096, keep=0.1, k=32, r=64, dtype="bf16"),
}


def config_shapes(name: str):
    cfg = CONFIGS[name]
    return [s for _ in range(cfg["layers"]) for s in cfg["shapes"]]


# ---------------------------------------------------------------------------
# torch backend (same recipe on any device; used where arrays only fit on the GPU)
# ---------------------------------------------------------------------------
def torch_gradients(spec: GradSpec, step: int, device, grad_dtype, want_mask: bool = True, anchor: bool = False):
    """One weight gradient (m x n) by the same recipe with torch ops on `device`, rounded to grad_dtype.

    anchor=False: masked gradient dY^T (X * Mk) / keep.  anchor=True: unmasked gradient of an independent batch.
    The contraction over tokens runs in fp32 (plain torch.matmul); the result is rounded once.
    """
    import torch
    gen = torch.Generator(device=device)
    k0, k1 = _key(spec, ((1 << 19) + step) if anchor else step, 0)
    gen.manual_seed((k0 * 0x9E3779B97F4A7C15 + k1) & 0x7FFFFFFFFFFFFFFF)
    T, m, n, k = spec.tokens, spec.m, spec.n, spec.planted_rank
    X = torch.randn((T, n), generator=gen, device=device, dtype=torch.float32)
    dY = torch.randn((T, m), generator=gen, device=device, dtype=torch.float32)
    if k > 0:
        pg = torch.Generator(device=device)
        pg.manual_seed(((int(spec.seed) * 1000003 + spec.layer) * 1000003 + spec.mat_id) & 0x7FFFFFFFFFFFFFFF)
        Px, _ = torch.linalg.qr(torch.randn((n, k), generator=pg, device=device, dtype=torch.float32))
        Py, _ = torch.linalg.qr(torch.randn((m, k), generator=pg, device=device, dtype=torch.float32))
        C = torch.randn((T, k), generator=gen, device=device, dtype=torch.float32)
        a = planted_amplitude(spec)
        X += a * (C @ Px.T)
        dY += a * (C @ Py.T)
    if (not anchor) and want_mask and spec.keep < 1.0:
        X *= (torch.rand((T, n), generator=gen, device=device) < spec.keep).to(torch.float32)
        X /= spec.keep
    return (dY.T @ X).to(grad_dtype)
