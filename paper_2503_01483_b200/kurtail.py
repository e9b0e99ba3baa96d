"""ctypes binding of libkurtail (argument marshalling only).

Every function here forwards to the C entry point of the same name declared in
include/kurtail.h; all arithmetic runs in the CUDA library.  torch is used for
device memory and streams only.  There is no fallback: if the shared library is
missing the import of this module's `lib()` raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# KURTAIL_LIB names another build of the same library (e.g. one compiled with other nvcc flags) to load instead
LIB_PATH = os.environ.get("KURTAIL_LIB") or os.path.join(_HERE, "libkurtail.so")

KT_BF16, KT_F32, KT_F64 = 0, 1, 2
STATUS = {0: "KT_OK", 1: "KT_ERR_INVALID_ARG", 2: "KT_ERR_SHAPE", 3: "KT_ERR_ALIGN", 4: "KT_ERR_WORKSPACE",
          5: "KT_ERR_ARCH", 6: "KT_ERR_CUDA", 7: "KT_ERR_NONFINITE", 8: "KT_ERR_TIMEOUT", 9: "KT_ERR_TOO_LARGE",
          10: "KT_ERR_COOPERATIVE", 11: "KT_ERR_REDUCE"}


class KtError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: {STATUS.get(status, status)}")


class kt_mat(C.Structure):
    _fields_ = [("data", C.c_void_p), ("dtype", C.c_int32), ("reserved", C.c_int32),
                ("rows", C.c_int64), ("cols", C.c_int64), ("ld", C.c_int64)]


class kt_config(C.Structure):
    _fields_ = [("kappa_target", C.c_float), ("cayley_iters", C.c_int32), ("q", C.c_float), ("eps", C.c_float),
                ("polish_thresh", C.c_float), ("retract_terms", C.c_int32), ("guard_every", C.c_int32),
                ("forward_terms", C.c_int32), ("small_d_fused", C.c_int32), ("small_d_orth", C.c_int32),
                ("optimizer", C.c_int32), ("beta1", C.c_float), ("beta2", C.c_float), ("adam_eps", C.c_float),
                ("norm_iters", C.c_int32), ("backward_mode", C.c_int32), ("cta_pairs", C.c_int32), ("loss_mode", C.c_int32), ("rmsnorm", C.c_int32), ("rms_eps", C.c_float),
                ("wait_limit_ms", C.c_int32), ("forward_bf16", C.c_int32)]


class kt_quant_spec(C.Structure):
    _fields_ = [("bits", C.c_int32), ("asymmetric", C.c_int32), ("clip", C.c_float), ("clip_mode", C.c_int32)]


class kt_adam_state(C.Structure):
    _fields_ = [("v", C.c_double), ("step", C.c_int32), ("reserved", C.c_int32)]


class kt_fit_report(C.Structure):
    _fields_ = [("steps_done", C.c_int32), ("degenerate_rows", C.c_int32), ("loss_first", C.c_double),
                ("loss_last", C.c_double), ("orth_err", C.c_double), ("alpha_last", C.c_float),
                ("w_norm_last", C.c_float), ("loss_history", C.POINTER(C.c_double)), ("w_op_last", C.c_float),
                ("series_terms_last", C.c_int32), ("p0_terms_last", C.c_int32), ("guards_run", C.c_int32)]


class kt_profile(C.Structure):
    _fields_ = [("launches_total", C.c_int64), ("gemm_launches", C.c_int32 * 8), ("gemm_ms", C.c_float * 8)]


EXPORTS = ["kt_default_config", "kt_create", "kt_destroy", "kt_status_string", "kt_workspace_bytes",
           "kt_set_workspace", "kt_init_rotation", "kt_kurtosis_loss", "kt_loss_grad", "kt_row_moments",
           "kt_rotate", "kt_orth_step", "kt_adam_step", "kt_orth_error", "kt_fit", "kt_fit_layers",
           "kt_fit_shared_workspace_bytes", "kt_fit_shared", "kt_fit_host", "kt_fit_sharded", "kt_fit_shared_sharded",
           "kt_test_wait_timeout",
           "kt_quant4_error", "kt_quant4_codes", "kt_quant_error", "kt_quant_codes", "kt_quant_error_given",
           "kt_rowmax_success", "kt_profile_begin", "kt_profile_end",
           "kt_kurtosis_loss_noalloc"]

# int32 reduce(void* user, void* dev_ptr, int64 count, int32 dtype, void* cuda_stream)
REDUCE_FN = C.CFUNCTYPE(C.c_int32, C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_void_p)

_lib = None


def lib():
    """Loads libkurtail.so (built by paper_2503_01483_b200.build).  Raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(f"{LIB_PATH} is missing: run `python -m paper_2503_01483_b200.build` "
                                "(there is no fallback path)")
    L = C.CDLL(LIB_PATH)
    vp, i32, i64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
    dp = C.POINTER(C.c_double)
    L.kt_default_config.argtypes = [C.POINTER(kt_config)]
    L.kt_default_config.restype = None
    L.kt_create.argtypes = [C.POINTER(vp), C.POINTER(kt_config), vp]
    L.kt_destroy.argtypes = [vp]
    L.kt_destroy.restype = None
    L.kt_status_string.argtypes = [i32]
    L.kt_status_string.restype = C.c_char_p
    L.kt_workspace_bytes.argtypes = [vp, i64, i64, i32, C.POINTER(C.c_size_t)]
    L.kt_set_workspace.argtypes = [vp, vp, C.c_size_t]
    L.kt_init_rotation.argtypes = [vp, vp, i64, i32]
    L.kt_kurtosis_loss.argtypes = [vp, kt_mat, vp, dp]
    L.kt_loss_grad.argtypes = [vp, kt_mat, vp, vp, dp]
    L.kt_row_moments.argtypes = [vp, kt_mat, vp, vp]
    L.kt_rotate.argtypes = [vp, kt_mat, vp, vp]
    L.kt_orth_step.argtypes = [vp, vp, vp, i64, f32]
    L.kt_adam_step.argtypes = [vp, vp, vp, vp, C.POINTER(kt_adam_state), i64, f32]
    L.kt_orth_error.argtypes = [vp, vp, i64, dp]
    L.kt_fit.argtypes = [vp, kt_mat, vp, i32, f32, C.POINTER(kt_fit_report)]
    L.kt_fit_layers.argtypes = [vp, C.POINTER(kt_mat), C.POINTER(vp), i32, i32, i32, f32, C.POINTER(kt_fit_report)]
    L.kt_fit_shared_workspace_bytes.argtypes = [vp, i64, i32, i64, C.POINTER(C.c_size_t)]
    L.kt_fit_shared.argtypes = [vp, C.POINTER(kt_mat), i32, i64, C.POINTER(i32), i32, vp, i32, f32,
                                C.POINTER(kt_fit_report)]
    L.kt_fit_host.argtypes = [vp, kt_mat, vp, vp, vp, i32, f32, C.POINTER(kt_fit_report)]
    L.kt_fit_sharded.argtypes = [vp, kt_mat, vp, i64, REDUCE_FN, vp, i32, f32, C.POINTER(kt_fit_report)]
    L.kt_fit_shared_sharded.argtypes = [vp, C.POINTER(kt_mat), i32, i64, C.POINTER(i32), i32, vp, i64, REDUCE_FN, vp,
                                        i32, f32, C.POINTER(kt_fit_report)]
    L.kt_test_wait_timeout.argtypes = [vp, i32]
    L.kt_quant4_error.argtypes = [vp, kt_mat, vp, dp]
    L.kt_quant4_codes.argtypes = [vp, vp, i64, i64, vp, vp]
    L.kt_quant_error.argtypes = [vp, kt_mat, vp, C.POINTER(kt_quant_spec), dp]
    L.kt_quant_codes.argtypes = [vp, vp, i64, i64, C.POINTER(kt_quant_spec), vp, vp, vp]
    L.kt_quant_error_given.argtypes = [vp, vp, i64, i64, C.POINTER(kt_quant_spec), dp]
    L.kt_rowmax_success.argtypes = [vp, kt_mat, vp, vp, dp]
    L.kt_kurtosis_loss_noalloc.argtypes = [kt_mat, vp, vp, vp]
    L.kt_profile_begin.argtypes = [vp]
    L.kt_profile_end.argtypes = [vp, C.POINTER(kt_profile)]
    for name in EXPORTS:
        fn = getattr(L, name)
        if name not in ("kt_default_config", "kt_destroy", "kt_status_string"):
            fn.restype = i32
    _lib = L
    return L


def default_config(**overrides):
    cfg = kt_config()
    lib().kt_default_config(C.byref(cfg))
    for k, v in overrides.items():
        setattr(cfg, k, v)
    return cfg


def _check(st, where):
    if st != 0:
        raise KtError(st, where)


def as_mat(X: torch.Tensor) -> kt_mat:
    """Describes a 2-D row-major torch tensor (bf16 or f32, device or host)."""
    if X.dim() != 2 or X.stride(1) != 1:
        raise ValueError("X must be 2-D with unit column stride")
    if X.dtype == torch.bfloat16:
        dt = KT_BF16
    elif X.dtype == torch.float32:
        dt = KT_F32
    else:
        raise ValueError("X must be bfloat16 or float32")
    return kt_mat(X.data_ptr(), dt, 0, X.shape[0], X.shape[1], X.stride(0))


def _rep_dict(rep, hist):
    return dict(steps_done=rep.steps_done, degenerate_rows=rep.degenerate_rows, loss_first=rep.loss_first,
                loss_last=rep.loss_last, orth_err=rep.orth_err, alpha_last=rep.alpha_last,
                w_norm_last=rep.w_norm_last, loss_history=list(hist) if hist is not None else None,
                w_op_last=rep.w_op_last, series_terms_last=rep.series_terms_last, p0_terms_last=rep.p0_terms_last,
                guards_run=rep.guards_run)


def kurtosis_loss_noalloc(X, R, loss_dev, stream=None):
    """kt_kurtosis_loss_noalloc: the loss without a context, a workspace or any allocation.
    `loss_dev` is a caller-owned float64 device tensor of one element; the call is stream
    ordered (synchronise before reading it).  Raises KtError(9) above N 16384 / d 1024."""
    sp = C.c_void_p(stream.cuda_stream if stream is not None else 0)
    with torch.cuda.device(X.device):     # the call works on the current device's copy of the built-in array
        _check(lib().kt_kurtosis_loss_noalloc(as_mat(X), R.data_ptr(), loss_dev.data_ptr(), sp),
               "kt_kurtosis_loss_noalloc")


class Context:
    """Owns a kt_ctx and (optionally) a torch-allocated workspace."""

    def __init__(self, device="cuda:0", stream=None, **cfg_overrides):
        self.device = torch.device(device)
        self.stream = stream
        self._ws = None
        self._ws_bytes = 0
        self._h = C.c_void_p()
        cfg = default_config(**cfg_overrides)
        with torch.cuda.device(self.device):
            sp = C.c_void_p(stream.cuda_stream if stream is not None else 0)
            _check(lib().kt_create(C.byref(self._h), C.byref(cfg), sp), "kt_create")

    def close(self):
        if self._h:
            lib().kt_destroy(self._h)
            self._h = C.c_void_p()
        self._ws = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- workspace --------------------------------------------------------
    def workspace_bytes(self, N, d, x_dtype=KT_BF16):
        n = C.c_size_t()
        _check(lib().kt_workspace_bytes(self._h, N, d, x_dtype, C.byref(n)), "kt_workspace_bytes")
        return n.value

    def ensure_workspace(self, N, d, x_dtype=KT_BF16):
        need = self.workspace_bytes(N, d, x_dtype)
        if need > self._ws_bytes:
            self._ws = None
            self._ws = torch.empty(need + 256, dtype=torch.uint8, device=self.device)
            base = (self._ws.data_ptr() + 255) // 256 * 256
            _check(lib().kt_set_workspace(self._h, C.c_void_p(base), need), "kt_set_workspace")
            self._ws_bytes = need

    def _prep(self, X):
        m = as_mat(X)
        self.ensure_workspace(m.rows, m.cols, m.dtype)
        return m

    # -- entry points (same names as the C ABI, without the kt_ prefix) -----
    def init_rotation(self, d, kind):
        R = torch.empty((d, d), dtype=torch.float32, device=self.device)
        k = {"identity": 0, "hadamard": 1}[kind] if isinstance(kind, str) else kind
        _check(lib().kt_init_rotation(self._h, R.data_ptr(), d, k), "kt_init_rotation")
        return R

    def kurtosis_loss(self, X, R):
        m = self._prep(X)
        out = C.c_double()
        _check(lib().kt_kurtosis_loss(self._h, m, R.data_ptr(), C.byref(out)), "kt_kurtosis_loss")
        return out.value

    def loss_grad(self, X, R, dR=None, want_loss=True):
        m = self._prep(X)
        if dR is None:
            dR = torch.empty_like(R)
        out = C.c_double()
        _check(lib().kt_loss_grad(self._h, m, R.data_ptr(), dR.data_ptr(), C.byref(out) if want_loss else None),
               "kt_loss_grad")
        return (out.value if want_loss else None), dR

    def row_moments(self, X, R):
        m = self._prep(X)
        mom = torch.empty((m.rows, 4), dtype=torch.float32, device=self.device)
        _check(lib().kt_row_moments(self._h, m, R.data_ptr(), mom.data_ptr()), "kt_row_moments")
        return mom

    def rotate(self, X, R):
        m = self._prep(X)
        Y = torch.empty((m.rows, m.cols), dtype=torch.float32, device=self.device)
        _check(lib().kt_rotate(self._h, m, R.data_ptr(), Y.data_ptr()), "kt_rotate")
        return Y

    def orth_step(self, R, dR, lr):
        d = R.shape[0]
        self.ensure_workspace(1, d, KT_BF16)
        _check(lib().kt_orth_step(self._h, R.data_ptr(), dR.data_ptr(), d, lr), "kt_orth_step")
        return R

    def adam_step(self, R, dR, M, state, lr):
        """kt_adam_step.  `state` is a dict(v=float, step=int), zero before the first step; updated in place."""
        d = R.shape[0]
        self.ensure_workspace(1, d, KT_BF16)
        st = kt_adam_state(float(state["v"]), int(state["step"]), 0)
        _check(lib().kt_adam_step(self._h, R.data_ptr(), dR.data_ptr(), M.data_ptr(), C.byref(st), d, lr),
               "kt_adam_step")
        state["v"], state["step"] = st.v, st.step
        return R

    def orth_error(self, R):
        d = R.shape[0]
        self.ensure_workspace(1, d, KT_BF16)
        out = C.c_double()
        _check(lib().kt_orth_error(self._h, R.data_ptr(), d, C.byref(out)), "kt_orth_error")
        return out.value

    def fit(self, X, R, steps, lr, history=False):
        m = self._prep(X)
        rep = kt_fit_report()
        hist = (C.c_double * max(steps, 1))() if history else None
        if history:
            rep.loss_history = C.cast(hist, C.POINTER(C.c_double))
        _check(lib().kt_fit(self._h, m, R.data_ptr(), steps, lr, C.byref(rep)), "kt_fit")
        return _rep_dict(rep, hist[:steps] if history else None)

    def fit_layers(self, Xs, Rs, steps, lr, first_layer=0):
        L = len(Xs)
        mats = (kt_mat * L)(*[as_mat(X) for X in Xs])
        self.ensure_workspace(mats[0].rows, mats[0].cols, mats[0].dtype)
        ptrs = (C.c_void_p * L)(*[R.data_ptr() for R in Rs])
        reps = (kt_fit_report * L)()
        _check(lib().kt_fit_layers(self._h, mats, ptrs, L, first_layer, steps, lr, reps), "kt_fit_layers")
        return [_rep_dict(r, None) for r in reps]

    def fit_shared(self, Xs, rows_per_sample, order, batch, R, steps, lr, history=False):
        """kt_fit_shared: one R for the equally shaped buffers Xs; `order` is a sequence of steps*batch sample ids."""
        nb = len(Xs)
        mats = (kt_mat * nb)(*[as_mat(X) for X in Xs])
        self._shared_workspace(rows_per_sample, batch, mats[0].cols)
        ids = (C.c_int32 * (steps * batch))(*[int(v) for v in order[:steps * batch]])
        rep = kt_fit_report()
        hist = (C.c_double * steps)() if history and steps > 0 else None
        if hist is not None:
            rep.loss_history = C.cast(hist, C.POINTER(C.c_double))
        _check(lib().kt_fit_shared(self._h, mats, nb, rows_per_sample, ids, batch, R.data_ptr(), steps, lr,
                                   C.byref(rep)), "kt_fit_shared")
        return _rep_dict(rep, hist)

    def _shared_workspace(self, rows_per_sample, batch, d):
        need = C.c_size_t()
        _check(lib().kt_fit_shared_workspace_bytes(self._h, rows_per_sample, batch, d, C.byref(need)),
               "kt_fit_shared_workspace_bytes")
        if need.value > self._ws_bytes:
            self._ws = None
            self._ws = torch.empty(need.value + 256, dtype=torch.uint8, device=self.device)
            base = (self._ws.data_ptr() + 255) // 256 * 256
            _check(lib().kt_set_workspace(self._h, C.c_void_p(base), need.value), "kt_set_workspace")
            self._ws_bytes = need.value

    def fit_sharded(self, X_local, R, rows_total, reduce, steps, lr, history=False):
        """kt_fit_sharded.  `reduce` is None (a single shard) or a Python callable
        reduce(dev_ptr, count, dtype, cuda_stream) -> 0 that enqueues an in-place sum all-reduce."""
        m = self._prep(X_local)
        rep = kt_fit_report()
        hist = (C.c_double * max(steps, 1))() if history else None
        if history:
            rep.loss_history = C.cast(hist, C.POINTER(C.c_double))
        cb = REDUCE_FN(lambda user, ptr, count, dtype, stream: int(reduce(ptr, count, dtype, stream))) \
            if reduce is not None else C.cast(None, REDUCE_FN)
        _check(lib().kt_fit_sharded(self._h, m, R.data_ptr(), rows_total, cb, None, steps, lr, C.byref(rep)),
               "kt_fit_sharded")
        return _rep_dict(rep, hist[:steps] if history else None)

    def fit_shared_sharded(self, Xs, rows_per_sample, order, batch, R, rows_total, reduce, steps, lr, history=False):
        """kt_fit_shared_sharded: this process's share (`batch` samples per step, its own `order`) of every minibatch."""
        nb = len(Xs)
        mats = (kt_mat * nb)(*[as_mat(X) for X in Xs])
        self._shared_workspace(rows_per_sample, batch, mats[0].cols)
        ids = (C.c_int32 * (steps * batch))(*[int(v) for v in order[:steps * batch]])
        rep = kt_fit_report()
        hist = (C.c_double * steps)() if history and steps > 0 else None
        if hist is not None:
            rep.loss_history = C.cast(hist, C.POINTER(C.c_double))
        cb = REDUCE_FN(lambda user, ptr, count, dtype, stream: int(reduce(ptr, count, dtype, stream))) \
            if reduce is not None else C.cast(None, REDUCE_FN)
        _check(lib().kt_fit_shared_sharded(self._h, mats, nb, rows_per_sample, ids, batch, R.data_ptr(), rows_total,
                                           cb, None, steps, lr, C.byref(rep)), "kt_fit_shared_sharded")
        return _rep_dict(rep, hist)

    def test_wait_timeout(self, limit_ms):
        _check(lib().kt_test_wait_timeout(self._h, limit_ms), "kt_test_wait_timeout")

    def fit_host(self, X_host, X_staging, R_host, R_dev, steps, lr):
        m = as_mat(X_host)
        self.ensure_workspace(m.rows, m.cols, m.dtype)
        rep = kt_fit_report()
        _check(lib().kt_fit_host(self._h, m, X_staging.data_ptr(), R_host.data_ptr(), R_dev.data_ptr(), steps, lr,
                                 C.byref(rep)), "kt_fit_host")
        return _rep_dict(rep, None)

    def quant4_error(self, X, R):
        m = self._prep(X)
        out = C.c_double()
        _check(lib().kt_quant4_error(self._h, m, R.data_ptr(), C.byref(out)), "kt_quant4_error")
        return out.value

    def quant_error(self, X, R, bits=4, asymmetric=False, clip=1.0, clip_mode=0):
        m = self._prep(X)
        spec = kt_quant_spec(bits, int(asymmetric), clip, clip_mode)
        out = C.c_double()
        _check(lib().kt_quant_error(self._h, m, R.data_ptr(), C.byref(spec), C.byref(out)), "kt_quant_error")
        return out.value

    def quant_codes(self, Y, bits=4, asymmetric=False, clip=1.0, clip_mode=0):
        N, d = Y.shape
        spec = kt_quant_spec(bits, int(asymmetric), clip, clip_mode)
        codes = torch.empty((N, d), dtype=torch.int16, device=Y.device)
        scales = torch.empty((N,), dtype=torch.float32, device=Y.device)
        shifts = torch.empty((N,), dtype=torch.float32, device=Y.device)
        _check(lib().kt_quant_codes(self._h, Y.data_ptr(), N, d, C.byref(spec), codes.data_ptr(), scales.data_ptr(),
                                    shifts.data_ptr()), "kt_quant_codes")
        return codes, scales, shifts

    def quant_error_given(self, Y, bits=4, asymmetric=False, clip=1.0, clip_mode=0):
        N, d = Y.shape
        self.ensure_workspace(N, max(128, (d + 127) // 128 * 128), KT_BF16)
        spec = kt_quant_spec(bits, int(asymmetric), clip, clip_mode)
        out = C.c_double()
        _check(lib().kt_quant_error_given(self._h, Y.data_ptr(), N, d, C.byref(spec), C.byref(out)),
               "kt_quant_error_given")
        return out.value

    def rowmax_success(self, X, R_a, R_b=None):
        m = self._prep(X)
        out = C.c_double()
        _check(lib().kt_rowmax_success(self._h, m, R_a.data_ptr(), R_b.data_ptr() if R_b is not None else None,
                                       C.byref(out)), "kt_rowmax_success")
        return out.value

    def profile_begin(self):
        _check(lib().kt_profile_begin(self._h), "kt_profile_begin")

    def profile_end(self):
        pr = kt_profile()
        _check(lib().kt_profile_end(self._h, C.byref(pr)), "kt_profile_end")
        names = ["forward", "backward_a", "backward_b", "square", "quant", "fused"]
        return dict(launches_total=pr.launches_total,
                    gemm={n: dict(launches=pr.gemm_launches[i], ms=pr.gemm_ms[i]) for i, n in enumerate(names)})

    def quant4_codes(self, Y):
        N, d = Y.shape
        codes = torch.empty((N, d), dtype=torch.int8, device=self.device)
        scales = torch.empty((N,), dtype=torch.float32, device=self.device)
        _check(lib().kt_quant4_codes(self._h, Y.data_ptr(), N, d, codes.data_ptr(), scales.data_ptr()),
               "kt_quant4_codes")
        return codes, scales
