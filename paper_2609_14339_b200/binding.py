"""ctypes binding of libspectral_correction.so: same names as the C ABI, argument marshalling only.

PyTorch is used for device memory and streams; every arithmetic step of the path runs in the library's
kernels.  There is no CPU fallback: if the library is missing or cannot be loaded, calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_NAME = "libspectral_correction.so"

SC_OK = 0
SC_WARN_NO_ANCHOR = 1
SC_DTYPE_BF16, SC_DTYPE_FP32 = 0, 1
SC_ENGINE_AUTO, SC_ENGINE_SIMT = 0, 1
SC_OPT_ADAMW, SC_OPT_ADEMAMIX = 0, 1


class SCError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s (%d)" % (where, status_string(status), status))


class Shape(C.Structure):
    _fields_ = [("rows", C.c_int64), ("cols", C.c_int64)]


class Hparams(C.Structure):
    """Mirror of sc_hparams."""
    _fields_ = [("alpha", C.c_float), ("tau_p", C.c_float), ("beta_anc", C.c_float), ("lr", C.c_float),
                ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float), ("weight_decay", C.c_float),
                ("max_grad_norm", C.c_float), ("grads_prescaled", C.c_int32), ("grad_dtype", C.c_int32),
                ("sketch_width", C.c_int32), ("power_iters", C.c_int32), ("engine", C.c_int32),
                ("collect_stats", C.c_int32), ("warm_start", C.c_int32), ("warm_power_iters", C.c_int32),
                ("optimizer", C.c_int32), ("seed", C.c_uint64), ("beta3", C.c_float), ("mix_alpha", C.c_float),
                ("full_spectrum", C.c_int32), ("fs_sqrt_iters", C.c_int32), ("fs_inv_iters", C.c_int32),
                ("reserved", C.c_int32)]

    @classmethod
    def default(cls, **kw) -> "Hparams":
        hp = cls()
        _check(load_library().sc_hparams_default(C.byref(hp)), "sc_hparams_default")
        for k, v in kw.items():
            if not hasattr(hp, k):
                raise AttributeError(k)
            setattr(hp, k, v)
        return hp


class OptState(C.Structure):
    _fields_ = [("exp_avg", C.POINTER(C.c_void_p)), ("exp_avg_sq", C.POINTER(C.c_void_p)),
                ("params_bf16", C.POINTER(C.c_void_p)), ("exp_avg_slow", C.POINTER(C.c_void_p))]


class Profile(C.Structure):
    _fields_ = [("ms", C.c_double * 6), ("spans", C.c_int64 * 6)]


PROFILE_CATEGORIES = ("anchor_ema", "basis_passes", "basis_small", "projection", "filter", "update")


class MatStats(C.Structure):
    _fields_ = [("g_sqnorm", C.c_float), ("x_sqnorm", C.c_float), ("gproj_sqnorm", C.c_float), ("r_eff", C.c_float)]


# every symbol include/spectral_correction.h declares: name -> (restype, argtypes)
_VP, _VPP = C.c_void_p, C.POINTER(C.c_void_p)
EXPORTS = {
    "sc_hparams_default": (C.c_int, [C.POINTER(Hparams)]),
    "sc_plan_workspace_bytes": (C.c_size_t, [C.POINTER(Shape), C.c_int, C.c_int, C.POINTER(Hparams)]),
    "sc_plan_create": (C.c_int, [C.POINTER(_VP), C.POINTER(Shape), C.c_int, C.c_int, C.c_float, C.POINTER(Hparams),
                                 _VP, C.c_size_t, _VP]),
    "sc_plan_destroy": (C.c_int, [_VP]),
    "sc_anchor_update": (C.c_int, [_VP, _VPP, C.c_int64]),
    "sc_anchor_update_factored": (C.c_int, [_VP, _VPP, _VPP, C.c_int, C.c_int64]),
    "sc_correct_and_step": (C.c_int, [_VP, _VPP, _VPP, C.POINTER(OptState), C.c_int64]),
    "sc_correct_and_step_host": (C.c_int, [_VP, _VPP, _VPP, _VPP, C.POINTER(OptState), C.c_int64, C.POINTER(MatStats),
                                           C.POINTER(C.c_float)]),
    "sc_apply_prf_mask": (C.c_int, [_VP, _VP, C.c_int64, C.c_int64, C.c_float, C.c_uint64, C.c_uint32, C.c_uint64, C.c_int,
                                    _VP]),
    "sc_masked_weight_grad": (C.c_int, [_VP, _VP, _VP, _VP, C.c_int, C.c_int64, C.c_int64, C.c_int64, C.c_float,
                                        C.c_uint64, C.c_uint32, C.c_uint64, _VP, _VP]),
    "sc_apply_prf_mask_exact_k": (C.c_int, [_VP, _VP, C.c_int64, C.c_int64, C.c_float, C.c_uint64, C.c_uint32, C.c_uint64,
                                            C.c_int, _VP]),
    "sc_lowrank_workspace_bytes": (C.c_size_t, [C.c_int64, C.c_int64, C.c_int]),
    "sc_lowrank_compress": (C.c_int, [_VP, C.c_int, _VP, _VP, _VP, C.c_int64, C.c_int64, C.c_int, C.c_int, _VP, C.c_size_t,
                                      _VP]),
    "sc_lowrank_init_q": (C.c_int, [_VP, C.c_int64, C.c_int, C.c_uint64, _VP]),
    "sc_export_basis": (C.c_int, [_VP, C.c_int, _VP, _VP, _VP]),
    "sc_import_basis": (C.c_int, [_VP, C.c_int, _VP, _VP, _VP]),
    "sc_export_projection": (C.c_int, [_VP, C.c_int, _VP, _VP]),
    "sc_project_static": (C.c_int, [_VP, C.c_int, _VP, _VP, C.c_int64, C.c_int64, C.c_int, _VP, _VP]),
    "sc_export_anchor_momentum": (C.c_int, [_VP, C.c_int, _VP]),
    "sc_import_anchor_momentum": (C.c_int, [_VP, C.c_int, _VP]),
    "sc_export_sketch": (C.c_int, [_VP, C.c_int64, C.c_int, _VP]),
    "sc_set_debug_gproj_out": (C.c_int, [_VP, _VPP]),
    "sc_get_stats": (C.c_int, [_VP, C.POINTER(MatStats), C.POINTER(C.c_float)]),
    "sc_get_device_status": (C.c_int, [_VP]),
    "sc_state_bytes": (C.c_size_t, [_VP]),
    "sc_state_export": (C.c_int, [_VP, _VP, C.c_size_t]),
    "sc_state_import": (C.c_int, [_VP, _VP, C.c_size_t]),
    "sc_debug_wait_probe": (C.c_int, [_VP, C.c_int]),
    "sc_set_profiling": (C.c_int, [_VP, C.c_int]),
    "sc_get_profile": (C.c_int, [_VP, C.POINTER(Profile)]),
    "sc_kernel_launch_count": (C.c_int64, []),
    "sc_get_anchor_info": (C.c_int, [_VP, C.POINTER(C.c_int64), C.POINTER(C.c_int)]),
    "sc_plan_uses_tensor_cores": (C.c_int, [_VP]),
    "sc_status_string": (C.c_char_p, [C.c_int]),
    "sc_version": (C.c_int, []),
}

_lib = None


def lib_path() -> str:
    return os.path.join(_HERE, _LIB_NAME)


def load_library():
    """dlopen the in-tree library and declare prototypes. Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise RuntimeError("%s is missing: run `python -m paper_2609_14339_b200.build` "
                           "(there is no CPU fallback)" % path)
    lib = C.CDLL(path)
    for name, (res, args) in EXPORTS.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().sc_status_string(int(status)).decode()


def _check(status: int, where: str, allow=(SC_OK,)) -> int:
    if status not in allow:
        raise SCError(status, where)
    return status


def _ptr_array(tensors: Optional[Sequence], n: int, allow_none: bool):
    if tensors is None:
        return None
    if len(tensors) != n:
        raise ValueError("expected %d tensors, got %d" % (n, len(tensors)))
    arr = (C.c_void_p * n)()
    for i, t in enumerate(tensors):
        if t is None:
            if not allow_none:
                raise ValueError("tensor %d is None" % i)
            arr[i] = None
        else:
            if not t.is_cuda or not t.is_contiguous():
                raise ValueError("tensor %d must be a contiguous CUDA tensor" % i)
            arr[i] = t.data_ptr()
    return arr


def project_static(G, U, V, X_out=None, stream=None):
    """X = U^T G V through sc_project_static: no plan, no workspace, no allocation inside the library.

    For callers that cannot allocate device memory where they need the projection (all of HBM already owned by
    a caching allocator, or a path that must not synchronise the device). G: rows x cols bf16/fp32, U: rows x r
    fp32, V: cols x r fp32, all contiguous CUDA tensors. Pass X_out (r x r fp32) to keep this wrapper from
    allocating too. Calls share one 8 MiB scratch array: do not let two of them overlap on the GPU.
    """
    import torch
    lib = load_library()
    rows, cols = G.shape
    r = U.shape[1]
    assert U.shape == (rows, r) and V.shape == (cols, r) and U.dtype == torch.float32 and V.dtype == torch.float32
    for t in (G, U, V):
        if not t.is_cuda or not t.is_contiguous():
            raise ValueError("tensors must be contiguous CUDA tensors")
    if X_out is None:
        X_out = torch.empty((r, r), dtype=torch.float32, device=G.device)
    dt = SC_DTYPE_BF16 if G.dtype == torch.bfloat16 else SC_DTYPE_FP32
    st = stream if stream is not None else torch.cuda.current_stream(G.device)
    with torch.cuda.device(G.device):
        _check(lib.sc_project_static(G.data_ptr(), dt, U.data_ptr(), V.data_ptr(), rows, cols, r, X_out.data_ptr(),
                                     st.cuda_stream), "sc_project_static")
    return X_out


def lowrank_init_q(cols: int, rho: int, seed: int, device="cuda:0", stream=None):
    """The +-1 start basis of the first compression step (cols x rho fp32)."""
    import torch
    lib = load_library()
    Q = torch.empty((cols, rho), dtype=torch.float32, device=device)
    st = stream if stream is not None else torch.cuda.current_stream(Q.device)
    with torch.cuda.device(Q.device):
        _check(lib.sc_lowrank_init_q(Q.data_ptr(), cols, rho, int(seed), st.cuda_stream), "sc_lowrank_init_q")
    return Q


def lowrank_compress(G, Q, E=None, P=None, phases: int = 7, workspace=None, stream=None):
    """One low-rank compression step with error feedback through sc_lowrank_compress.

    G: rows x cols bf16/fp32; Q: cols x rho fp32 (in: previous Q, out: new Q); E: rows x cols fp32 error memory
    (updated in place) or None; P: rows x rho fp32 (allocated when None). Returns (P, Q, workspace)."""
    import torch
    lib = load_library()
    rows, cols = G.shape
    rho = Q.shape[1]
    assert Q.shape == (cols, rho) and Q.dtype == torch.float32 and Q.is_contiguous() and G.is_contiguous()
    if P is None:
        P = torch.empty((rows, rho), dtype=torch.float32, device=G.device)
    assert P.shape == (rows, rho) and P.dtype == torch.float32 and P.is_contiguous()
    if E is not None:
        assert E.shape == (rows, cols) and E.dtype == torch.float32 and E.is_contiguous()
    need = lib.sc_lowrank_workspace_bytes(rows, cols, rho)
    if need == 0:
        raise SCError(-1, "sc_lowrank_workspace_bytes")
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=G.device)
    dt = SC_DTYPE_BF16 if G.dtype == torch.bfloat16 else SC_DTYPE_FP32
    st = stream if stream is not None else torch.cuda.current_stream(G.device)
    with torch.cuda.device(G.device):
        _check(lib.sc_lowrank_compress(G.data_ptr(), dt, E.data_ptr() if E is not None else None, P.data_ptr(),
                                       Q.data_ptr(), rows, cols, rho, int(phases), workspace.data_ptr(),
                                       workspace.numel(), st.cuda_stream), "sc_lowrank_compress")
    return P, Q, workspace


def masked_weight_grad(dY, X, keep: float, seed: int, layer: int, step: int, out_dtype=None, Xm=None, out=None,
                       status=None, stream=None):
    """G = dY^T (X * M(seed, layer, step)) / keep for one linear layer: the mask pass and a tensor-core GEMM over the
    tokens. dY: tokens x rows, X: tokens x cols, both bf16 on the GPU. Returns (G, Xm); Xm holds X * M (unscaled)."""
    import torch
    lib = load_library()
    assert dY.is_cuda and X.is_cuda and dY.is_contiguous() and X.is_contiguous()
    assert dY.dtype == torch.bfloat16 and X.dtype == torch.bfloat16 and dY.dim() == 2 and X.dim() == 2
    assert dY.shape[0] == X.shape[0]
    tokens, rows, cols = X.shape[0], dY.shape[1], X.shape[1]
    out_dtype = torch.bfloat16 if out_dtype is None else out_dtype
    if Xm is None:
        Xm = torch.empty_like(X)
    if out is None:
        out = torch.empty((rows, cols), device=X.device, dtype=out_dtype)
    assert out.is_contiguous() and out.shape == (rows, cols) and out.dtype in (torch.bfloat16, torch.float32)
    st = stream if stream is not None else torch.cuda.current_stream(X.device)
    with torch.cuda.device(X.device):
        _check(lib.sc_masked_weight_grad(dY.data_ptr(), X.data_ptr(), Xm.data_ptr(), out.data_ptr(),
                                         0 if out.dtype == torch.bfloat16 else 1, tokens, rows, cols, float(keep),
                                         int(seed), int(layer), int(step),
                                         status.data_ptr() if status is not None else None, st.cuda_stream),
               "sc_masked_weight_grad")
    return out, Xm


def apply_prf_mask(X, keep: float, seed: int, layer: int, step: int, rescale: bool = True, out=None, stream=None,
                   exact_k: bool = False):
    """h~ = h * M(seed, layer, step) (/ keep): the shared-PRF activation mask, bf16 tokens x features on the GPU.
    exact_k=True keeps exactly round(keep * features) features per token instead of independent coin flips."""
    import torch
    lib = load_library()
    if exact_k:
        assert X.is_cuda and X.is_contiguous() and X.dtype == torch.bfloat16 and X.dim() == 2
        if out is None:
            out = torch.empty_like(X)
        st = stream if stream is not None else torch.cuda.current_stream(X.device)
        with torch.cuda.device(X.device):
            _check(lib.sc_apply_prf_mask_exact_k(X.data_ptr(), out.data_ptr(), X.shape[0], X.shape[1], float(keep),
                                                 int(seed), int(layer), int(step), int(bool(rescale)), st.cuda_stream),
                   "sc_apply_prf_mask_exact_k")
        return out
    assert X.is_cuda and X.is_contiguous() and X.dtype == torch.bfloat16 and X.dim() == 2
    if out is None:
        out = torch.empty_like(X)
    st = stream if stream is not None else torch.cuda.current_stream(X.device)
    with torch.cuda.device(X.device):
        _check(lib.sc_apply_prf_mask(X.data_ptr(), out.data_ptr(), X.shape[0], X.shape[1], float(keep), int(seed),
                                     int(layer), int(step), int(bool(rescale)), st.cuda_stream), "sc_apply_prf_mask")
    return out


class Plan:
    """Owns a workspace tensor and an sc_plan handle; methods mirror the C entry points one to one."""

    def __init__(self, shapes, rank: int, keep_ratio: float, hp: Optional[Hparams] = None, stream=None, device="cuda:0",
                 workspace=None):
        """workspace: optional caller-owned uint8 CUDA tensor of at least workspace_bytes(...) bytes whose data pointer
        is 256-byte aligned; by default the plan allocates one."""
        import torch
        self._torch = torch
        self.lib = load_library()
        self.hp = hp if hp is not None else Hparams.default()
        self.shapes = [(int(m), int(n)) for m, n in shapes]
        self.n_mats = len(self.shapes)
        self.rank = int(rank)
        self.device = torch.device(device)
        arr = (Shape * self.n_mats)(*[Shape(m, n) for m, n in self.shapes])
        need = self.lib.sc_plan_workspace_bytes(arr, self.n_mats, self.rank, C.byref(self.hp))
        if need == 0:
            raise SCError(-1, "sc_plan_workspace_bytes")
        self.workspace_bytes = int(need)
        with torch.cuda.device(self.device):
            if workspace is not None:
                if workspace.dtype != torch.uint8 or not workspace.is_cuda or workspace.numel() < need:
                    raise ValueError("workspace must be a uint8 CUDA tensor of at least %d bytes" % need)
                self.workspace = workspace
                base = workspace.data_ptr()
            else:
                self.workspace = torch.empty(need + 256, dtype=torch.uint8, device=self.device)
                base = (self.workspace.data_ptr() + 255) // 256 * 256
            self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
            handle = C.c_void_p()
            _check(self.lib.sc_plan_create(C.byref(handle), arr, self.n_mats, self.rank, float(keep_ratio),
                                           C.byref(self.hp), base, need, self.stream.cuda_stream), "sc_plan_create")
        self.handle = handle
        self._keep = []

    @staticmethod
    def workspace_bytes_for(shapes, rank: int, hp: Optional[Hparams] = None) -> int:
        lib = load_library()
        hp = hp if hp is not None else Hparams.default()
        arr = (Shape * len(shapes))(*[Shape(int(m), int(n)) for m, n in shapes])
        return int(lib.sc_plan_workspace_bytes(arr, len(shapes), int(rank), C.byref(hp)))

    def close(self):
        if getattr(self, "handle", None):
            self.lib.sc_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the three calls of the method -------------------------------------------------------------
    def anchor_update(self, anchor_grads: Sequence, step_tag: int) -> int:
        arr = _ptr_array(anchor_grads, self.n_mats, True)
        return _check(self.lib.sc_anchor_update(self.handle, arr, int(step_tag)), "sc_anchor_update")

    def anchor_update_factored(self, P_factors: Sequence, Q_factors: Sequence, step_tag: int) -> int:
        rho = next(t.shape[1] for t in P_factors if t is not None)
        return _check(self.lib.sc_anchor_update_factored(self.handle, _ptr_array(P_factors, self.n_mats, True),
                                                         _ptr_array(Q_factors, self.n_mats, True), int(rho),
                                                         int(step_tag)), "sc_anchor_update_factored")

    def correct_and_step(self, masked_grads, params, exp_avg, exp_avg_sq, step: int, params_bf16=None,
                         exp_avg_slow=None) -> int:
        """exp_avg_slow: the slow EMA of the dual-EMA optimizer (required when hp.optimizer is SC_OPT_ADEMAMIX)."""
        n = self.n_mats
        st = OptState(_ptr_array(exp_avg, n, False), _ptr_array(exp_avg_sq, n, False),
                      _ptr_array(params_bf16, n, True) if params_bf16 is not None else None,
                      _ptr_array(exp_avg_slow, n, False) if exp_avg_slow is not None else None)
        return _check(self.lib.sc_correct_and_step(self.handle, _ptr_array(masked_grads, n, False),
                                                   _ptr_array(params, n, False), C.byref(st), int(step)),
                      "sc_correct_and_step", allow=(SC_OK, SC_WARN_NO_ANCHOR))

    def correct_and_step_host(self, host_grads, grad_staging, params, exp_avg, exp_avg_sq, step: int, params_bf16=None,
                              want_stats: bool = True, exp_avg_slow=None):
        """Gradients in host tensors (pin them for overlap); returns (status, stats or None, clip)."""
        n = self.n_mats
        harr = (C.c_void_p * n)()
        for i, t in enumerate(host_grads):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError("host gradient %d must be a contiguous CPU tensor" % i)
            harr[i] = t.data_ptr()
        st = OptState(_ptr_array(exp_avg, n, False), _ptr_array(exp_avg_sq, n, False),
                      _ptr_array(params_bf16, n, True) if params_bf16 is not None else None,
                      _ptr_array(exp_avg_slow, n, False) if exp_avg_slow is not None else None)
        stats = (MatStats * n)() if want_stats else None
        clip = C.c_float(1.0)
        rc = _check(self.lib.sc_correct_and_step_host(self.handle, harr, _ptr_array(grad_staging, n, False),
                                                      _ptr_array(params, n, False), C.byref(st), int(step), stats,
                                                      C.byref(clip)),
                    "sc_correct_and_step_host", allow=(SC_OK, SC_WARN_NO_ANCHOR))
        out = None
        if stats is not None:
            out = [dict(g_sqnorm=a.g_sqnorm, x_sqnorm=a.x_sqnorm, gproj_sqnorm=a.gproj_sqnorm, r_eff=a.r_eff) for a in stats]
        return rc, out, clip.value

    # ---- inspection --------------------------------------------------------------------------------
    def export_basis(self, mat: int):
        t = self._torch
        m, n = self.shapes[mat]
        r = self.rank
        U = t.empty((m, r), dtype=t.float32, device=self.device)
        s = t.empty((r,), dtype=t.float32, device=self.device)
        V = t.empty((n, r), dtype=t.float32, device=self.device)
        if r > 0:
            _check(self.lib.sc_export_basis(self.handle, mat, U.data_ptr(), s.data_ptr(), V.data_ptr()), "sc_export_basis")
        return U, s, V

    def import_basis(self, mat: int, U, s, V):
        t = self._torch
        U = U.to(self.device, t.float32).contiguous(); s = s.to(self.device, t.float32).contiguous()
        V = V.to(self.device, t.float32).contiguous()
        m, n = self.shapes[mat]
        assert U.shape == (m, self.rank) and V.shape == (n, self.rank) and s.shape == (self.rank,)
        _check(self.lib.sc_import_basis(self.handle, mat, U.data_ptr(), s.data_ptr(), V.data_ptr()), "sc_import_basis")
        self._torch.cuda.current_stream(self.device).wait_stream(self.stream)
        self.stream.synchronize()

    def export_projection(self, mat: int):
        t = self._torch
        m, n = self.shapes[mat]
        T = t.empty((m, self.rank), dtype=t.float32, device=self.device)
        X = t.empty((self.rank, self.rank), dtype=t.float32, device=self.device)
        if self.rank > 0:
            _check(self.lib.sc_export_projection(self.handle, mat, T.data_ptr(), X.data_ptr()), "sc_export_projection")
        return T, X

    def export_anchor_momentum(self, mat: int):
        t = self._torch
        M = t.empty(self.shapes[mat], dtype=t.float32, device=self.device)
        _check(self.lib.sc_export_anchor_momentum(self.handle, mat, M.data_ptr()), "sc_export_anchor_momentum")
        return M

    def import_anchor_momentum(self, mat: int, M):
        M = M.to(self.device, self._torch.float32).contiguous()
        assert tuple(M.shape) == self.shapes[mat]
        _check(self.lib.sc_import_anchor_momentum(self.handle, mat, M.data_ptr()), "sc_import_anchor_momentum")
        self.stream.synchronize()

    def export_sketch(self, rows: int, width: int):
        t = self._torch
        Om = t.empty((rows, width), dtype=t.float32, device=self.device)
        _check(self.lib.sc_export_sketch(self.handle, rows, width, Om.data_ptr()), "sc_export_sketch")
        return Om

    def set_debug_gproj_out(self, tensors):
        self._keep = list(tensors) if tensors is not None else []
        arr = _ptr_array(tensors, self.n_mats, True) if tensors is not None else None
        _check(self.lib.sc_set_debug_gproj_out(self.handle, arr), "sc_set_debug_gproj_out")

    def get_stats(self):
        arr = (MatStats * self.n_mats)()
        clip = C.c_float()
        _check(self.lib.sc_get_stats(self.handle, arr, C.byref(clip)), "sc_get_stats")
        return [dict(g_sqnorm=a.g_sqnorm, x_sqnorm=a.x_sqnorm, gproj_sqnorm=a.gproj_sqnorm, r_eff=a.r_eff)
                for a in arr], clip.value

    def get_device_status(self) -> int:
        return int(self.lib.sc_get_device_status(self.handle))

    def get_anchor_info(self):
        tag, k = C.c_int64(), C.c_int()
        _check(self.lib.sc_get_anchor_info(self.handle, C.byref(tag), C.byref(k)), "sc_get_anchor_info")
        return tag.value, k.value

    def state_export(self):
        """Anchor momentum + cached basis of every matrix as one bytes-like host buffer (a ctypes array)."""
        n = self.lib.sc_state_bytes(self.handle)
        buf = (C.c_char * n)()
        _check(self.lib.sc_state_export(self.handle, buf, n), "sc_state_export")
        return buf

    def state_import(self, buf):
        _check(self.lib.sc_state_import(self.handle, buf, len(buf)), "sc_state_import")

    def debug_wait_probe(self, max_polls: int = 4096):
        _check(self.lib.sc_debug_wait_probe(self.handle, int(max_polls)), "sc_debug_wait_probe")

    def set_profiling(self, on: bool):
        _check(self.lib.sc_set_profiling(self.handle, int(bool(on))), "sc_set_profiling")

    def get_profile(self):
        pr = Profile()
        _check(self.lib.sc_get_profile(self.handle, C.byref(pr)), "sc_get_profile")
        return {name: dict(ms=pr.ms[i], spans=pr.spans[i]) for i, name in enumerate(PROFILE_CATEGORIES)}

    def uses_tensor_cores(self) -> bool:
        return bool(self.lib.sc_plan_uses_tensor_cores(self.handle))
