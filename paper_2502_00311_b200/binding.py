"""Thin ctypes binding of the C-ABI library declared in include/sgc.h (argument marshalling only).

PyTorch supplies device memory and streams; every step of the path runs inside the CUDA library.
The library must have been built (paper_2502_00311_b200.build.build()); loading fails loudly otherwise.
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libsgc_b200.so")
_lib = None

EXPORTS = ["sgc_create", "sgc_step", "sgc_step_group", "sgc_step_chunked", "sgc_cesgc_step", "sgc_destroy", "sgc_set_alpha", "sgc_get", "sgc_set_state",
           "sgc_clear_status", "sgc_last_launches", "sgc_set_profile", "sgc_get_profile", "sgc_sparsify_static", "sgc_z_block",
           "sgc_set_mode", "sgc_set_recovery", "sgc_screen", "sgc_reproject", "sgc_strerror", "sgc_version", "sgc_status",
           "sgc_set_wait_limit", "sgc_set_max_rounds"]

# selectors of sgc_get: name -> (code, dtype, length attribute or None for a scalar)
RECORDS = dict(t=(0, np.int64, None), M=(1, np.float32, "k"), V=(2, np.float32, "k"), sel_idx=(3, np.uint32, "s"),
               sel_val=(4, np.float32, "s"), p=(5, np.float64, "k"), q=(6, np.float64, "k"),
               lamM=(7, np.uint32, "s"), lamV=(8, np.uint32, "s"), xM=(9, np.float64, "s"), xV=(10, np.float64, "s"),
               upd_idx=(11, np.uint32, "s"), upd_val=(12, np.float64, "s"), n_upd=(13, np.int32, None),
               status=(14, np.uint32, None), mismatch=(15, np.int32, None), negv=(16, np.int32, None),
               doneM=(17, np.int32, None), doneV=(18, np.int32, None), rnormM=(19, np.float64, "s"),
               rnormV=(20, np.float64, "s"), rounds=(21, np.int32, None), fallback=(22, np.int32, None),
               n_cand=(23, np.int32, None), round_trace=(24, np.int32, 72), list_rounds=(25, np.int32, None),
               pass_rows=(26, np.int32, None))

MODE_AUTO, MODE_LOCKSTEP, MODE_SPECULATIVE = 0, 1, 2

STATUS_NONFINITE_INPUT = 1
STATUS_DEPENDENT_COLUMN = 2
STATUS_SUPPORT_MISMATCH = 4
STATUS_NEGATIVE_V = 8
STATUS_CANDIDATE_OVERFLOW = 16
STATUS_SELECT_FALLBACK = 32
STATUS_TIMEOUT = 64


class SgcError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__("%s failed with code %d: %s" % (where, code, strerror(code)))


def lib():
    """Loads the shared library once; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError("CUDA library %s is missing: run paper_2502_00311_b200.build.build() "
                               "(there is no CPU fallback)" % _LIB_PATH)
        L = C.CDLL(_LIB_PATH)
        vp = C.c_void_p
        L.sgc_create.restype = C.c_int
        L.sgc_create.argtypes = [C.POINTER(vp), C.c_int64, C.c_int32, C.c_int32, C.c_uint64, C.c_float, C.c_float,
                                 C.c_float, C.c_float]
        L.sgc_step.restype = C.c_int
        L.sgc_step.argtypes = [vp, vp, vp, vp]
        L.sgc_step_group.restype = C.c_int
        L.sgc_step_group.argtypes = [C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.c_int32, vp]
        L.sgc_step_chunked.restype = C.c_int
        L.sgc_step_chunked.argtypes = [C.POINTER(vp), C.c_int32, vp, vp, vp]
        L.sgc_cesgc_step.restype = C.c_int
        L.sgc_cesgc_step.argtypes = [C.POINTER(vp), C.c_int32, vp, C.c_int32, C.c_int32, C.c_int32, vp, vp, vp, vp]
        L.sgc_destroy.restype = C.c_int
        L.sgc_destroy.argtypes = [vp]
        L.sgc_set_alpha.restype = C.c_int
        L.sgc_set_alpha.argtypes = [vp, C.c_float]
        L.sgc_get.restype = C.c_int
        L.sgc_get.argtypes = [vp, C.c_int32, vp, C.c_size_t]
        L.sgc_set_state.restype = C.c_int
        L.sgc_set_state.argtypes = [vp, vp, vp, C.c_int64]
        L.sgc_clear_status.restype = C.c_int
        L.sgc_clear_status.argtypes = [vp]
        L.sgc_status.restype = C.c_int
        L.sgc_status.argtypes = [vp, C.POINTER(C.c_uint32)]
        L.sgc_set_wait_limit.restype = C.c_int
        L.sgc_set_wait_limit.argtypes = [vp, C.c_uint64]
        L.sgc_set_max_rounds.restype = C.c_int
        L.sgc_set_max_rounds.argtypes = [vp, C.c_int32]
        L.sgc_last_launches.restype = C.c_int
        L.sgc_last_launches.argtypes = [vp, C.POINTER(C.c_int32)]
        L.sgc_set_profile.restype = C.c_int
        L.sgc_set_profile.argtypes = [vp, C.c_int]
        L.sgc_get_profile.restype = C.c_int
        L.sgc_get_profile.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(C.c_int32)]
        L.sgc_sparsify_static.restype = C.c_int
        L.sgc_sparsify_static.argtypes = [vp, C.c_int64, C.c_int32, vp, vp, vp, vp]
        L.sgc_z_block.restype = C.c_int
        L.sgc_z_block.argtypes = [C.c_uint64, C.c_int64, C.c_int64, C.c_int64, C.c_int64, vp, vp]
        L.sgc_set_mode.restype = C.c_int
        L.sgc_set_mode.argtypes = [vp, C.c_int32]
        L.sgc_set_recovery.restype = C.c_int
        L.sgc_set_recovery.argtypes = [vp, C.c_int32, C.c_double]
        L.sgc_reproject.restype = C.c_int
        L.sgc_reproject.argtypes = [vp, C.c_uint64, vp]
        L.sgc_screen.restype = C.c_int
        L.sgc_screen.argtypes = [C.c_uint64, C.c_int64, C.c_int32, C.c_int32, vp, vp, vp, vp, C.c_int32, vp, vp]
        L.sgc_strerror.restype = C.c_char_p
        L.sgc_strerror.argtypes = [C.c_int]
        L.sgc_version.restype = C.c_int
        L.sgc_version.argtypes = []
        _lib = L
    return _lib


def strerror(code):
    return lib().sgc_strerror(int(code)).decode()


def version():
    return int(lib().sgc_version())


def _check(rc, where):
    if rc != 0:
        raise SgcError(rc, where)


def set_screen_wait_limit(ns):
    """Bound (ns) of the waits inside the pass that sgc_screen launches; 0 restores the default."""
    _check(lib().sgc_set_wait_limit(None, C.c_uint64(int(ns))), "sgc_set_wait_limit")


def _dev_ptr(t, n, what):
    """Device pointer of a contiguous float32 CUDA tensor with at least n elements."""
    import torch
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
        raise TypeError("%s must be a contiguous float32 CUDA tensor" % what)
    if t.numel() < n:
        raise ValueError("%s has %d elements, need %d" % (what, t.numel(), n))
    return C.c_void_p(t.data_ptr())


def _stream_ptr(stream):
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def z_block(seed, row0, nrows, col0, ncols, stream=None):
    """Z(seed, row, col) for a block as a float32 CUDA tensor [nrows, ncols] (sgc_z_block)."""
    import torch
    out = torch.empty((nrows, ncols), dtype=torch.float32, device="cuda")
    _check(lib().sgc_z_block(C.c_uint64(seed), row0, nrows, col0, ncols, C.c_void_p(out.data_ptr()),
                             _stream_ptr(stream)), "sgc_z_block")
    return out


def screen(seed, d, k, rt, tau, rep_cap, stream=None):
    """sgc_screen: tensor-core screening pass.  rt: CUDA int16/uint16-sized tensor [n, k] of binary16 bit patterns
    (or a torch.float16 tensor), tau: float32 CUDA tensor [n].  Returns (rep_count [n] int32, rep [n, rep_cap, 2] int32
    holding (column, score bits), error_flag [1] int32) as CUDA tensors; nothing is synchronised."""
    import torch
    n = rt.shape[0]
    if rt.element_size() != 2 or not rt.is_cuda or not rt.is_contiguous() or rt.shape[1] != k:
        raise TypeError("rt must be a contiguous CUDA tensor [n, k] of 16-bit elements")
    rep_count = torch.empty(n, dtype=torch.int32, device="cuda")
    rep = torch.empty((n, rep_cap, 2), dtype=torch.int32, device="cuda")
    err = torch.empty(1, dtype=torch.int32, device="cuda")
    _check(lib().sgc_screen(C.c_uint64(seed), int(d), int(k), int(n), C.c_void_p(rt.data_ptr()), _dev_ptr(tau, n, "tau"),
                            C.c_void_p(rep_count.data_ptr()), C.c_void_p(rep.data_ptr()), int(rep_cap),
                            C.c_void_p(err.data_ptr()), _stream_ptr(stream)), "sgc_screen")
    return rep_count, rep, err


def sparsify_static(grad, s, out_idx, out_val, out_status=None, stream=None):
    """sgc_sparsify_static: top-s selection into caller-provided CUDA tensors, without any device allocation.

    For hosts that cannot call cudaMalloc when they need the selection (all device memory already handed to a
    framework's pool, or a thread that must not trigger cudaMalloc's device-wide synchronisation).  out_idx:
    int32/uint32-sized CUDA tensor of s elements, out_val: float32 CUDA tensor of s elements, out_status:
    optional CUDA tensor holding one 32-bit word.  Calls on one device share a static scratch array inside the
    library and must not overlap on the GPU.
    """
    d = grad.numel()
    if out_idx.numel() < s or out_idx.element_size() != 4 or not out_idx.is_cuda or not out_idx.is_contiguous():
        raise TypeError("out_idx must be a contiguous CUDA tensor of at least s 32-bit integers")
    st_ptr = C.c_void_p(out_status.data_ptr()) if out_status is not None else C.c_void_p(0)
    _check(lib().sgc_sparsify_static(_dev_ptr(grad, d, "grad"), d, int(s), C.c_void_p(out_idx.data_ptr()),
                                     _dev_ptr(out_val, s, "out_val"), st_ptr, _stream_ptr(stream)),
           "sgc_sparsify_static")


class Sgc:
    """One SGC optimizer state (sgc_create / sgc_step / sgc_destroy)."""

    def __init__(self, d, k, s, seed, lr, beta1, beta2, eps, alpha=None):
        self.d, self.k, self.s = int(d), int(k), int(s)
        h = C.c_void_p()
        _check(lib().sgc_create(C.byref(h), self.d, self.k, self.s, C.c_uint64(seed), lr, beta1, beta2, eps),
               "sgc_create")
        self._h = h
        if alpha is not None:
            self.set_alpha(alpha)

    def set_mode(self, mode):
        _check(lib().sgc_set_mode(self._h, int(mode)), "sgc_set_mode")

    def set_recovery(self, shared_support, residual_tol=0.0):
        """Opt-in variant: one support (that of OMP_A(M^)) for both moments, and / or an early stop on ||r||."""
        _check(lib().sgc_set_recovery(self._h, 1 if shared_support else 0, float(residual_tol)), "sgc_set_recovery")

    def reproject(self, new_seed, stream=None):
        """SGCA: switch to the matrix named by new_seed and re-align M, V with it (after the step of an iteration t = 0 mod T)."""
        _check(lib().sgc_reproject(self._h, C.c_uint64(new_seed), _stream_ptr(stream)), "sgc_reproject")

    def set_alpha(self, alpha):
        _check(lib().sgc_set_alpha(self._h, alpha), "sgc_set_alpha")

    def step(self, grad, weight, stream=None):
        _check(lib().sgc_step(self._h, _dev_ptr(grad, self.d, "grad"), _dev_ptr(weight, self.d, "weight"),
                              _stream_ptr(stream)), "sgc_step")

    def get(self, name):
        code, dt, dim = RECORDS[name]
        n = 1 if dim is None else (dim if isinstance(dim, int) else getattr(self, dim))
        out = np.empty(n, dtype=dt)
        _check(lib().sgc_get(self._h, code, out.ctypes.data_as(C.c_void_p), out.nbytes), "sgc_get(%s)" % name)
        return out[0] if dim is None else out

    def set_state(self, M, V, t):
        M = np.ascontiguousarray(M, dtype=np.float32)
        V = np.ascontiguousarray(V, dtype=np.float32)
        if M.size != self.k or V.size != self.k:
            raise ValueError("M and V must have k elements")
        _check(lib().sgc_set_state(self._h, M.ctypes.data_as(C.c_void_p), V.ctypes.data_as(C.c_void_p), int(t)),
               "sgc_set_state")

    def status(self):
        out = C.c_uint32(0)
        _check(lib().sgc_status(self._h, C.byref(out)), "sgc_status")
        return out.value

    def set_wait_limit(self, ns):
        """Bound (ns) of the waits inside this state's screening passes; 0 restores the default."""
        _check(lib().sgc_set_wait_limit(self._h, C.c_uint64(int(ns))), "sgc_set_wait_limit")

    def set_max_rounds(self, rounds):
        """Most speculation rounds a step enqueues (what they leave open is finished in lock-step); 0 = automatic."""
        _check(lib().sgc_set_max_rounds(self._h, C.c_int32(int(rounds))), "sgc_set_max_rounds")

    def clear_status(self):
        _check(lib().sgc_clear_status(self._h), "sgc_clear_status")

    def last_launches(self):
        n = C.c_int32(0)
        _check(lib().sgc_last_launches(self._h, C.byref(n)), "sgc_last_launches")
        return n.value

    def set_profile(self, enable):
        _check(lib().sgc_set_profile(self._h, 1 if enable else 0), "sgc_set_profile")

    def get_profile(self):
        """Per-phase totals since set_profile(True): dict phase -> (ms, launches)."""
        ms = (C.c_float * 8)()
        n = (C.c_int32 * 8)()
        _check(lib().sgc_get_profile(self._h, ms, n), "sgc_get_profile")
        names = ("select_sample", "select_filter", "select_pick", "project_adam", "omp", "resolve", "scatter", "pass")
        return {names[i]: (float(ms[i]), int(n[i])) for i in range(8)}

    def close(self):
        if getattr(self, "_h", None):
            h, self._h = self._h, None
            _check(lib().sgc_destroy(h), "sgc_destroy")

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Mesgc:
    """Memory-efficient SGC (Section 4.4): c chunks of one flat vector, each with its own optimizer state and
    s_c entries per step, all sharing the matrix A (k x d/c) named by one seed (sgc_step_chunked)."""

    def __init__(self, d, c, k, s_c, seed, lr, beta1, beta2, eps, alpha=None):
        if d % c:
            raise ValueError("d must be a multiple of the number of chunks")
        self.d, self.c = int(d), int(c)
        self.chunks = [Sgc(d // c, k, s_c, seed, lr, beta1, beta2, eps, alpha=alpha) for _ in range(c)]
        self._hs = (C.c_void_p * self.c)(*[st._h for st in self.chunks])       # the handle array of every call

    def step(self, grad, weight, stream=None):
        _check(lib().sgc_step_chunked(self._hs, self.c, _dev_ptr(grad, self.d, "grad"), _dev_ptr(weight, self.d, "weight"),
                                      _stream_ptr(stream)), "sgc_step_chunked")

    def close(self):
        for st in self.chunks:
            st.close()


class Cesgc:
    """Compute-efficient SGC (Section 4.4): SGC, chunked, on the projected gradient B G of an m x n matrix; the update
    returns through B^T (sgc_cesgc_step).  B (r x m, float32, CUDA, orthonormal rows: the paper takes the leading left-singular
    vectors of a gradient and renews them every fixed number of iterations) is the caller's: set_projection() stores it."""

    def __init__(self, m, n, r, c, k, s_c, seed, lr, beta1, beta2, eps, alpha=None):
        import torch
        if (r * n) % c:
            raise ValueError("r * n must be a multiple of the number of chunks")
        self.m, self.n, self.r, self.c = int(m), int(n), int(r), int(c)
        self.core = Mesgc(r * n, c, k, s_c, seed, lr, beta1, beta2, eps, alpha=alpha)
        self.scratch = torch.empty(2 * r * n, dtype=torch.float32, device="cuda")
        self.B = None

    def set_projection(self, B):
        if B.shape != (self.r, self.m) or not B.is_cuda or not B.is_contiguous() or B.element_size() != 4:
            raise TypeError("B must be a contiguous float32 CUDA tensor of shape (r, m)")
        self.B = B

    def step(self, grad, weight, stream=None):
        if self.B is None:
            raise ValueError("set_projection() first")
        d = self.m * self.n
        _check(lib().sgc_cesgc_step(self.core._hs, self.c, C.c_void_p(self.B.data_ptr()), self.r, self.m, self.n,
                                    _dev_ptr(grad, d, "grad"), _dev_ptr(weight, d, "weight"),
                                    C.c_void_p(self.scratch.data_ptr()), _stream_ptr(stream)), "sgc_cesgc_step")

    def close(self):
        self.core.close()


def step_group(states, grads, weights, stream=None):
    """sgc_step_group: one step for several states that share (d, k, s, seed)."""
    n = len(states)
    if not (n == len(grads) == len(weights)) or n == 0:
        raise ValueError("states, grads and weights must be non-empty lists of equal length")
    hs = (C.c_void_p * n)(*[st._h for st in states])
    gs = (C.c_void_p * n)(*[_dev_ptr(g, states[i].d, "grad") for i, g in enumerate(grads)])
    ws = (C.c_void_p * n)(*[_dev_ptr(w, states[i].d, "weight") for i, w in enumerate(weights)])
    _check(lib().sgc_step_group(hs, gs, ws, n, _stream_ptr(stream)), "sgc_step_group")
