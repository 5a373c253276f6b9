"""Thin ctypes binding of libdeflpolar.so: argument marshalling only.

Every function has the name and meaning of the C entry point declared in include/defl.h. Tensors
are torch CUDA tensors used purely as device memory; all computation happens in the library's
CUDA kernels. There is no fallback: if the shared library is missing the import of this module's
`lib()` fails, and without a CUDA device every compute call raises.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdeflpolar.so")

BF16, F32, F16 = 0, 1, 2
RESTORE_PADDED, RESTORE_ADD = 0, 1
NORM_LANCZOS, NORM_FROBENIUS = 0, 1
ENGINE_AUTO, ENGINE_SIMT, ENGINE_TENSOR = 0, 1, 2
ST_CHOL_SHIFT, ST_JACOBI_CAP, ST_ZERO_RESIDUAL, ST_DEVICE_WAIT, ST_NONFINITE = 1, 2, 4, 8, 16
MAX_L, MAX_STEPS, MAX_TERMS = 64, 32, 6

MUON_QUINTIC = (3.4445, -4.7750, 2.0315)
CLASSICAL_QUINTIC = (1.875, -1.25, 0.375)

EXPORTS = [
    "defl_create", "defl_destroy", "defl_set_stream", "defl_polar_workspace_bytes", "defl_psd_workspace_bytes",
    "defl_polar_window", "defl_psd_window", "defl_polar_batched", "defl_polar_batched_host", "defl_muon_step_batched", "defl_brsvd_batched", "defl_psd_project", "defl_inv_root", "defl_admm_diag_sdp", "defl_fill_gaussian", "defl_debug_gemm",
    "defl_frobenius_norms_noalloc", "defl_set_profiling", "defl_get_stage_ms", "defl_get_stage_ms_sum", "defl_launch_count", "defl_device_wait_status",
    "defl_status_string", "defl_last_error",
]


class DeflOpts(ctypes.Structure):
    _fields_ = [("sketch", ctypes.c_void_p), ("seed", ctypes.c_uint64), ("restore_mode", ctypes.c_int),
                ("gamma", ctypes.c_float), ("norm_mode", ctypes.c_int), ("lanczos_start", ctypes.c_void_p),
                ("warmup", ctypes.c_int), ("engine", ctypes.c_int), ("exploit_symmetry", ctypes.c_int),
                ("tau", ctypes.c_float), ("half_filter", ctypes.c_int), ("bf16_iterates", ctypes.c_int),
                ("poly_terms", ctypes.c_int)]


class DeflInfo(ctypes.Structure):
    _fields_ = [("s", ctypes.c_void_p), ("rho", ctypes.c_void_p), ("status", ctypes.c_void_p),
                ("k_used", ctypes.c_void_p)]


_lib = None


def lib():
    """Load the shared library (raises OSError if it has not been built)."""
    global _lib
    if _lib is None:
        L = ctypes.CDLL(LIB_PATH)
        L.defl_create.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.c_int]
        L.defl_destroy.argtypes = [ctypes.c_void_p]
        L.defl_set_stream.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
        L.defl_polar_workspace_bytes.restype = ctypes.c_size_t
        L.defl_polar_workspace_bytes.argtypes = [ctypes.c_int] * 6
        L.defl_psd_workspace_bytes.restype = ctypes.c_size_t
        L.defl_psd_workspace_bytes.argtypes = [ctypes.c_int] * 2
        L.defl_polar_window.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_float, ctypes.c_float,
                                        ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_int)]
        L.defl_psd_window.argtypes = [ctypes.c_int, ctypes.c_float, ctypes.c_float,
                                      ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_int)]
        L.defl_polar_batched.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p] + [ctypes.c_int] * 7 + [
            ctypes.POINTER(ctypes.c_float), ctypes.c_int, ctypes.POINTER(DeflOpts), ctypes.POINTER(DeflInfo)]
        L.defl_polar_batched_host.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p] + [ctypes.c_int] * 7 + [
            ctypes.POINTER(ctypes.c_float), ctypes.c_int, ctypes.POINTER(DeflOpts)]
        L.defl_muon_step_batched.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p] + [
            ctypes.c_int] * 4 + [ctypes.c_float, ctypes.c_float, ctypes.c_int, ctypes.c_float, ctypes.c_float] + [
            ctypes.c_int] * 3 + [ctypes.POINTER(ctypes.c_float), ctypes.c_int, ctypes.POINTER(DeflOpts), ctypes.POINTER(DeflInfo)]
        L.defl_brsvd_batched.argtypes = [ctypes.c_void_p, ctypes.c_void_p] + [ctypes.c_int] * 7 + [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(DeflOpts), ctypes.c_void_p]
        L.defl_psd_project.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                                       ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(ctypes.c_float), ctypes.c_int,
                                       ctypes.POINTER(DeflOpts), ctypes.POINTER(DeflInfo)]
        L.defl_inv_root.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                    ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.POINTER(DeflOpts),
                                    ctypes.POINTER(DeflInfo)]
        L.defl_admm_diag_sdp.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_float,
                                         ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                         ctypes.c_int, ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(ctypes.c_float),
                                         ctypes.c_int, ctypes.POINTER(DeflOpts), ctypes.POINTER(ctypes.c_float)]
        L.defl_fill_gaussian.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_uint64]
        L.defl_debug_gemm.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                      ctypes.c_void_p, ctypes.c_longlong, ctypes.c_longlong, ctypes.c_longlong,
                                      ctypes.c_void_p, ctypes.c_longlong, ctypes.c_longlong, ctypes.c_longlong,
                                      ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_float, ctypes.c_int]
        L.defl_set_profiling.argtypes = [ctypes.c_void_p, ctypes.c_int]
        L.defl_get_stage_ms.argtypes = [ctypes.c_void_p, ctypes.POINTER(ctypes.c_float), ctypes.c_int]
        L.defl_get_stage_ms_sum.argtypes = [ctypes.c_void_p, ctypes.POINTER(ctypes.c_float), ctypes.c_int, ctypes.c_int]
        L.defl_launch_count.restype = ctypes.c_longlong
        L.defl_launch_count.argtypes = [ctypes.c_void_p]
        L.defl_device_wait_status.argtypes = [ctypes.c_void_p, ctypes.c_int]
        L.defl_status_string.restype = ctypes.c_char_p
        L.defl_status_string.argtypes = [ctypes.c_int]
        L.defl_last_error.restype = ctypes.c_char_p
        L.defl_last_error.argtypes = [ctypes.c_void_p]
        _lib = L
    return _lib


class DeflError(RuntimeError):
    def __init__(self, code, detail=""):
        self.code = code
        msg = lib().defl_status_string(code).decode()
        super().__init__("defl error %d: %s%s" % (code, msg, (" [" + detail + "]") if detail else ""))


def _dtype_code(t):
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.float16:
        return F16
    raise TypeError("only bfloat16, float16 and float32 tensors are supported")


def _ptr(t):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else None


def _dev(t, what):
    if not (t.is_cuda and t.is_contiguous()):
        raise ValueError("%s must be a contiguous CUDA tensor" % what)
    return t


def _schedule(coeffs, steps=None, terms=3):
    """[L][terms] coefficients as a C float array: one tuple repeated `steps` times, or a list of tuples."""
    c = torch.as_tensor(coeffs, dtype=torch.float64)
    if c.ndim == 1:
        c = c.unsqueeze(0).repeat(steps, 1)
    if c.numel() and c.shape[1] != terms:
        raise ValueError("every filter step takes %d coefficients, got %d" % (terms, c.shape[1]))
    flat = [float(x) for x in c.reshape(-1).tolist()]
    arr = (ctypes.c_float * max(len(flat), 1))(*flat)
    return arr, c.shape[0]


def defl_polar_window(m, n, w, delta):
    """(k, oversample) from the paper's ratios: k = ceil(w min(m,n)), oversample = min(min(m,n), k + ceil(delta min(m,n))) - k."""
    k, p = ctypes.c_int(), ctypes.c_int()
    rc = lib().defl_polar_window(m, n, w, delta, ctypes.byref(k), ctypes.byref(p))
    if rc != 0:
        raise DeflError(rc)
    return k.value, p.value


def defl_psd_window(n, w, w_prime):
    """(k, K) from the paper's ratios: k = ceil(w n), K = ceil(w' n)."""
    k, K = ctypes.c_int(), ctypes.c_int()
    rc = lib().defl_psd_window(n, w, w_prime, ctypes.byref(k), ctypes.byref(K))
    if rc != 0:
        raise DeflError(rc)
    return k.value, K.value


class Context:
    """defl_ctx bound to one CUDA device; work is enqueued on torch's current stream at call time."""

    def __init__(self, device=0):
        self.device = torch.device("cuda", device) if not isinstance(device, torch.device) else device
        h = ctypes.c_void_p()
        rc = lib().defl_create(ctypes.byref(h), self.device.index or 0)
        if rc != 0:
            raise DeflError(rc)
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            lib().defl_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _sync_stream(self):
        s = torch.cuda.current_stream(self.device)
        lib().defl_set_stream(self._h, ctypes.c_void_p(s.cuda_stream))

    def _check(self, rc):
        if rc != 0:
            raise DeflError(rc, lib().defl_last_error(self._h).decode())

    def _opts(self, sketch=None, seed=0, restore_mode=RESTORE_PADDED, gamma=0.0, norm_mode=NORM_LANCZOS,
              lanczos_start=None, warmup=False, engine=ENGINE_AUTO, exploit_symmetry=False, tau=0.0, half_filter=False, bf16_iterates=False,
              poly_terms=0):
        o = DeflOpts()
        o.sketch = sketch.data_ptr() if sketch is not None else None
        o.seed = seed
        o.restore_mode = restore_mode
        o.gamma = gamma
        o.norm_mode = norm_mode
        o.lanczos_start = lanczos_start.data_ptr() if lanczos_start is not None else None
        o.warmup = int(bool(warmup))
        o.engine = engine
        o.exploit_symmetry = int(bool(exploit_symmetry))
        o.tau = tau
        o.half_filter = int(bool(half_filter))
        o.bf16_iterates = int(bf16_iterates)      # 0 mixed (default), 1 / True bf16 throughout, 2 half throughout
        o.poly_terms = int(poly_terms)            # 0 / 3 quintic steps, 2 cubic, 4.. the higher-degree maps of Eq. 5
        return o

    # ------------------------------------------------------------------------------------------
    def defl_polar_batched(self, G, k, oversample, power_iters, coeff_schedule, steps=None, out=None, sketch=None,
                           seed=0, restore_mode=RESTORE_PADDED, gamma=0.0, engine=ENGINE_AUTO,
                           exploit_symmetry=False, want_info=False, tau=0.0, bf16_iterates=False, poly_terms=0):
        """out[b,m,n] = deflated polar factor of every G[b] (Algorithm 3 + Algorithm 1). poly_terms: coefficients per
        filter step (0 or 3: quintic; 4: the degree-seven map of Eq. 5, ...)."""
        _dev(G, "G")
        if G.ndim != 3:
            raise ValueError("G must be [b, m, n]")
        b, m, n = G.shape
        out = torch.empty_like(G) if out is None else _dev(out, "out")
        sched, L = _schedule(coeff_schedule, steps, poly_terms or 3)
        if sketch is not None:
            _dev(sketch, "sketch")
            if sketch.dtype != torch.float32:
                raise TypeError("sketch must be float32")
        opts = self._opts(sketch=sketch, seed=seed, restore_mode=restore_mode, gamma=gamma, engine=engine,
                          exploit_symmetry=exploit_symmetry, tau=tau, bf16_iterates=bf16_iterates, poly_terms=poly_terms)
        info = DeflInfo()
        extras = None
        if want_info:
            l = min(min(m, n), k + oversample) if k > 0 else 0
            s = torch.zeros((b, max(l, 1)), dtype=torch.float32, device=G.device)
            rho = torch.zeros((b,), dtype=torch.float32, device=G.device)
            status = torch.zeros((b,), dtype=torch.int32, device=G.device)
            k_used = torch.zeros((b,), dtype=torch.int32, device=G.device)
            info.s, info.rho, info.status = s.data_ptr(), rho.data_ptr(), status.data_ptr()
            info.k_used = k_used.data_ptr()
            extras = {"s": s[:, :l], "rho": rho, "status": status, "k_used": k_used}
        self._sync_stream()
        rc = lib().defl_polar_batched(self._h, _ptr(G), _ptr(out), b, m, n, _dtype_code(G), k, oversample, power_iters,
                                      sched, L, ctypes.byref(opts), ctypes.byref(info))
        self._check(rc)
        return (out, extras) if want_info else out

    def defl_muon_step_batched(self, W, Mom, Grad, lr, mu, k, oversample, power_iters, coeff_schedule, steps=None,
                               nesterov=False, weight_decay=0.0, scale=1.0, sketch=None, seed=0,
                               restore_mode=RESTORE_PADDED, gamma=0.0, engine=ENGINE_AUTO, exploit_symmetry=False,
                               tau=0.0):
        """One Deflated Muon step on a shape group, in place: Mom <- mu Mom + Grad (Grad may be None),
        W <- (1 - lr wd) W - lr scale F(Mom or its Nesterov look-ahead), F = defl_polar_batched's map."""
        _dev(W, "W"), _dev(Mom, "Mom")
        if Mom.ndim != 3 or W.shape != Mom.shape:
            raise ValueError("W and Mom must be [b, m, n] of the same shape")
        if Grad is not None:
            _dev(Grad, "Grad")
            if Grad.shape != Mom.shape or Grad.dtype != Mom.dtype:
                raise ValueError("Grad must match Mom in shape and type")
        b, m, n = Mom.shape
        sched, L = _schedule(coeff_schedule, steps)
        if sketch is not None:
            _dev(sketch, "sketch")
            if sketch.dtype != torch.float32:
                raise TypeError("sketch must be float32")
        opts = self._opts(sketch=sketch, seed=seed, restore_mode=restore_mode, gamma=gamma, engine=engine,
                          exploit_symmetry=exploit_symmetry, tau=tau)
        self._sync_stream()
        rc = lib().defl_muon_step_batched(self._h, _ptr(W), _dtype_code(W), _ptr(Mom), _ptr(Grad) if Grad is not None else None,
                                          b, m, n, _dtype_code(Mom), lr, mu, int(bool(nesterov)), weight_decay, scale,
                                          k, oversample, power_iters, sched, L, ctypes.byref(opts), None)
        self._check(rc)
        return W

    def defl_polar_batched_host(self, G_host, out_host, k, oversample, power_iters, coeff_schedule, steps=None,
                                sketch=None, seed=0, restore_mode=RESTORE_PADDED, gamma=0.0, engine=ENGINE_AUTO,
                                exploit_symmetry=False):
        """Host-buffer form: G_host/out_host are CPU tensors (pinned for speed); returns when out_host is filled."""
        if G_host.is_cuda or out_host.is_cuda or not (G_host.is_contiguous() and out_host.is_contiguous()):
            raise ValueError("G_host and out_host must be contiguous CPU tensors")
        b, m, n = G_host.shape
        sched, L = _schedule(coeff_schedule, steps)
        opts = self._opts(sketch=sketch, seed=seed, restore_mode=restore_mode, gamma=gamma, engine=engine,
                          exploit_symmetry=exploit_symmetry)
        self._sync_stream()
        rc = lib().defl_polar_batched_host(self._h, ctypes.c_void_p(G_host.data_ptr()),
                                           ctypes.c_void_p(out_host.data_ptr()), b, m, n, _dtype_code(G_host), k,
                                           oversample, power_iters, sched, L, ctypes.byref(opts))
        self._check(rc)
        return out_host

    def defl_brsvd_batched(self, G, k, oversample, power_iters, sketch=None, seed=0, engine=ENGINE_AUTO):
        """Algorithm 3 in the caller's orientation: returns (P[b,m,l], s[b,l], W[b,n,l], status[b])."""
        _dev(G, "G")
        b, m, n = G.shape
        l = min(min(m, n), k + oversample)
        P = torch.empty((b, m, l), dtype=torch.float32, device=G.device)
        W = torch.empty((b, n, l), dtype=torch.float32, device=G.device)
        s = torch.empty((b, l), dtype=torch.float32, device=G.device)
        status = torch.zeros((b,), dtype=torch.int32, device=G.device)
        opts = self._opts(sketch=sketch, seed=seed, engine=engine)
        self._sync_stream()
        rc = lib().defl_brsvd_batched(self._h, _ptr(G), b, m, n, _dtype_code(G), k, oversample, power_iters,
                                      _ptr(P), _ptr(s), _ptr(W), ctypes.byref(opts), _ptr(status))
        self._check(rc)
        return P, s, W, status

    def defl_psd_project(self, X, k, warm_basis, coeff_schedule, steps=None, out=None, gamma=0.0,
                         norm_mode=NORM_LANCZOS, lanczos_start=None, seed=0, warmup=False, engine=ENGINE_AUTO,
                         exploit_symmetry=False, want_info=False, tau=0.0, half_filter=False):
        """P = deflated PSD projection of the symmetric X[n,n] (Algorithm 2); warm_basis[n,K] is updated in place."""
        _dev(X, "X")
        n = X.shape[0]
        if X.dtype != torch.float32 or X.shape != (n, n):
            raise ValueError("X must be a square float32 matrix")
        K = 0
        if warm_basis is not None:
            _dev(warm_basis, "warm_basis")
            K = warm_basis.shape[1]
        out = torch.empty_like(X) if out is None else _dev(out, "out")
        sched, T = _schedule(coeff_schedule, steps)
        opts = self._opts(gamma=gamma, norm_mode=norm_mode, lanczos_start=lanczos_start, seed=seed, warmup=warmup,
                          engine=engine, exploit_symmetry=exploit_symmetry, tau=tau, half_filter=half_filter)
        info = DeflInfo()
        extras = None
        if want_info:
            lam = torch.zeros((max(K, 1),), dtype=torch.float32, device=X.device)
            theta = torch.zeros((1,), dtype=torch.float32, device=X.device)
            status = torch.zeros((1,), dtype=torch.int32, device=X.device)
            k_used = torch.zeros((1,), dtype=torch.int32, device=X.device)
            info.s, info.rho, info.status = lam.data_ptr(), theta.data_ptr(), status.data_ptr()
            info.k_used = k_used.data_ptr()
            extras = {"lam": lam[:K], "theta": theta, "status": status, "k_used": k_used}
        self._sync_stream()
        rc = lib().defl_psd_project(self._h, _ptr(X), _ptr(out), n, k, _ptr(warm_basis), K, sched, T,
                                    ctypes.byref(opts), ctypes.byref(info))
        self._check(rc)
        return (out, extras) if want_info else out

    def defl_inv_root(self, A, p, k, warm_basis, steps, out=None, gamma=0.0, norm_mode=NORM_LANCZOS, lanczos_start=None,
                      seed=0, warmup=False, engine=ENGINE_AUTO, exploit_symmetry=False, want_info=False, tau=0.0):
        """out ~ A^(-1/p) for the symmetric positive definite A[n,n]: deflation of the k leading eigenpairs tracked by
        warm_basis[n,K] (updated in place) around `steps` coupled Newton steps (Conclusion's next instance)."""
        _dev(A, "A")
        n = A.shape[0]
        if A.dtype != torch.float32 or A.shape != (n, n):
            raise ValueError("A must be a square float32 matrix")
        K = 0
        if warm_basis is not None:
            _dev(warm_basis, "warm_basis")
            K = warm_basis.shape[1]
        out = torch.empty_like(A) if out is None else _dev(out, "out")
        opts = self._opts(gamma=gamma, norm_mode=norm_mode, lanczos_start=lanczos_start, seed=seed, warmup=warmup,
                          engine=engine, exploit_symmetry=exploit_symmetry, tau=tau)
        info = DeflInfo()
        extras = None
        if want_info:
            lam = torch.zeros((max(K, 1),), dtype=torch.float32, device=A.device)
            theta = torch.zeros((1,), dtype=torch.float32, device=A.device)
            status = torch.zeros((1,), dtype=torch.int32, device=A.device)
            k_used = torch.zeros((1,), dtype=torch.int32, device=A.device)
            info.s, info.rho, info.status = lam.data_ptr(), theta.data_ptr(), status.data_ptr()
            info.k_used = k_used.data_ptr()
            extras = {"lam": lam[:K], "theta": theta, "status": status, "k_used": k_used}
        self._sync_stream()
        rc = lib().defl_inv_root(self._h, _ptr(A), _ptr(out), n, int(p), int(k), _ptr(warm_basis), K, int(steps),
                                 ctypes.byref(opts), ctypes.byref(info))
        self._check(rc)
        return (out, extras) if want_info else out

    def defl_admm_diag_sdp(self, C, b, sigma, iters, X, S, k, warm_basis, coeff_schedule, steps=None, warmup_iters=0,
                           gamma=0.0, norm_mode=NORM_LANCZOS, lanczos_start=None, seed=0, engine=ENGINE_AUTO,
                           exploit_symmetry=False, tau=0.0, half_filter=False):
        """`iters` ADMM iterations for min <C,X> s.t. diag(X) = b, X PSD (Appendix E.1, "ADMM for Standard-Form SDP"), X and S updated in place.
        Returns (y[n], residuals[iters,3]) with the three eigenvalue-free KKT terms per iteration."""
        _dev(C, "C"), _dev(b, "b"), _dev(X, "X"), _dev(S, "S")
        n = C.shape[0]
        for t, nm in ((C, "C"), (X, "X"), (S, "S")):
            if t.dtype != torch.float32 or tuple(t.shape) != (n, n):
                raise ValueError(nm + " must be a float32 [n, n] matrix")
        if b.dtype != torch.float32 or tuple(b.shape) != (n,):
            raise ValueError("b must be a float32 [n] vector")
        K = 0
        if warm_basis is not None:
            _dev(warm_basis, "warm_basis")
            K = warm_basis.shape[1]
        sched, T = _schedule(coeff_schedule, steps)
        opts = self._opts(gamma=gamma, norm_mode=norm_mode, lanczos_start=lanczos_start, seed=seed, engine=engine,
                          exploit_symmetry=exploit_symmetry, tau=tau, half_filter=half_filter)
        y = torch.zeros((n,), dtype=torch.float32, device=C.device)
        res = (ctypes.c_float * max(3 * iters, 1))()
        self._sync_stream()
        rc = lib().defl_admm_diag_sdp(self._h, _ptr(C), _ptr(b), n, sigma, iters, warmup_iters, _ptr(X), _ptr(S), _ptr(y),
                                      k, _ptr(warm_basis), K, sched, T, ctypes.byref(opts), res)
        self._check(rc)
        return y, torch.tensor(list(res)[:3 * iters], dtype=torch.float32).reshape(iters, 3)

    def defl_fill_gaussian(self, dst, seed):
        _dev(dst, "dst")
        self._sync_stream()
        self._check(lib().defl_fill_gaussian(self._h, _ptr(dst), dst.numel(), _dtype_code(dst), seed))
        return dst

    def defl_debug_gemm(self, A, B, trans_a=False, trans_b=False, engine=ENGINE_AUTO, out_dtype=None, alpha=1.0,
                        exploit_symmetry=False, transpose_out=False, withhold_first_step=False):
        """C[b] = alpha * op(A[b]) op(B[b]); op = transpose of the stored matrix when the flag is set. With
        transpose_out the engine writes the product transposed: the result has shape [b, N, M]."""
        _dev(A, "A"), _dev(B, "B")
        b = A.shape[0]
        if trans_a:
            K, M = A.shape[1], A.shape[2]
            sa_i, sa_k = 1, M
        else:
            M, K = A.shape[1], A.shape[2]
            sa_i, sa_k = K, 1
        if trans_b:
            N = B.shape[1]
            sb_k, sb_j = 1, B.shape[2]
        else:
            N = B.shape[2]
            sb_k, sb_j = N, 1
        out_dtype = out_dtype or A.dtype
        C = torch.empty((b, N, M) if transpose_out else (b, M, N), dtype=out_dtype, device=A.device)
        self._sync_stream()
        rc = lib().defl_debug_gemm(self._h, engine, b, M, N, K, _ptr(A), sa_i, sa_k, A.shape[1] * A.shape[2],
                                   _ptr(B), sb_k, sb_j, B.shape[1] * B.shape[2], _ptr(C), _dtype_code(A),
                                   {torch.bfloat16: BF16, torch.float16: F16}.get(out_dtype, F32), alpha,
                                   int(bool(exploit_symmetry)) | (2 if transpose_out else 0) | (4 if withhold_first_step else 0))
        self._check(rc)
        return C

    def defl_set_profiling(self, enabled):
        lib().defl_set_profiling(self._h, int(bool(enabled)))

    def defl_get_stage_ms(self, ncalls=1):
        """Stage durations (ms) of the last call, or their sums over the last `ncalls` calls; synchronises."""
        buf = (ctypes.c_float * 16)()
        n = lib().defl_get_stage_ms_sum(self._h, buf, 16, int(ncalls))
        return [buf[i] for i in range(max(n, 0))]

    def defl_launch_count(self):
        return int(lib().defl_launch_count(self._h))

    def defl_device_wait_status(self, clear=True):
        """The tensor engine's wait word (DEFL_ST_DEVICE_WAIT if a bounded device-side wait ran out); synchronises."""
        rc = lib().defl_device_wait_status(self._h, int(bool(clear)))
        if rc < 0:
            self._check(rc)
        return rc

    def polar_workspace_bytes(self, b, m, n, dtype, k, oversample):
        return int(lib().defl_polar_workspace_bytes(b, m, n, BF16 if dtype == torch.bfloat16 else F32, k, oversample))
