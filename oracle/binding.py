"""ctypes binding of the CPU oracle (oracle/sgc_oracle.cpp).  Test infrastructure only.

The shared object is compiled on first use with g++ (no CUDA involved) next to the source.
Every wrapper takes and returns numpy arrays; the arithmetic lives in the C++ file.
"""
import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sgc_oracle.cpp")
_SO = os.path.join(_HERE, "libsgc_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force=False):
    """Compile the oracle into oracle/libsgc_oracle.so (rebuilds when the source is newer)."""
    if (not force) and os.path.exists(_SO) and os.path.getmtime(_SO) >= os.path.getmtime(_SRC):
        return _SO
    tmp = _SO + ".tmp%d" % os.getpid()
    cmd = ["g++", "-O3", "-std=c++17", "-fopenmp", "-ffp-contract=off", "-mavx2", "-mfma", "-shared", "-fPIC",
           _SRC, "-o", tmp]
    subprocess.check_call(cmd)
    os.replace(tmp, _SO)
    return _SO


def lib():
    global _lib
    with _lock:
        if _lib is None:
            L = C.CDLL(build())
            u32p, f32p, f64p, i32p = (C.POINTER(C.c_uint32), C.POINTER(C.c_float), C.POINTER(C.c_double),
                                      C.POINTER(C.c_int32))
            L.orc_sigma.restype = C.c_float
            L.orc_sigma.argtypes = [C.c_int32]
            L.orc_z_block.restype = None
            L.orc_z_block.argtypes = [C.c_uint64, C.c_int64, C.c_int64, C.c_int64, C.c_int64, f32p]
            L.orc_half_round.restype = C.c_uint16
            L.orc_half_round.argtypes = [C.c_double]
            L.orc_half_value.restype = C.c_double
            L.orc_half_value.argtypes = [C.c_uint16]
            L.orc_half_fma.restype = C.c_uint16
            L.orc_half_fma.argtypes = [C.c_uint16, C.c_uint16, C.c_uint16]
            L.orc_half_mul.restype = C.c_uint16
            L.orc_half_mul.argtypes = [C.c_uint16, C.c_uint16]
            L.orc_z_of_byte_sum.restype = C.c_uint16
            L.orc_z_of_byte_sum.argtypes = [C.c_int32]
            L.orc_sparsify.restype = C.c_int32
            L.orc_sparsify.argtypes = [f32p, C.c_int64, C.c_int32, u32p, f32p]
            L.orc_project.restype = None
            L.orc_project.argtypes = [C.c_uint64, C.c_int32, u32p, f32p, C.c_int32, f64p, f64p]
            L.orc_adam.restype = None
            L.orc_adam.argtypes = [f32p, f32p, f64p, f64p, C.c_int32, C.c_float, C.c_float, C.c_int64, f64p, f64p]
            L.orc_omp.restype = C.c_int32
            L.orc_omp.argtypes = [C.c_uint64, C.c_int64, C.c_int32, C.c_int32, f64p, u32p, f64p, f64p, f64p, f64p]
            L.orc_omp_tol.restype = C.c_int32
            L.orc_omp_tol.argtypes = [C.c_uint64, C.c_int64, C.c_int32, C.c_int32, f64p, C.c_double, u32p, f64p, f64p, f64p,
                                      f64p]
            L.orc_select.restype = None
            L.orc_select.argtypes = [C.c_uint64, C.c_int64, C.c_int32, C.c_int32, f64p, u32p, i32p, C.c_int32,
                                     C.POINTER(C.c_int64), f64p, f64p]
            L.orc_least_squares.restype = C.c_int32
            L.orc_least_squares.argtypes = [C.c_uint64, C.c_int32, u32p, C.c_int32, f64p, f64p]
            L.orc_set_recovery.restype = None
            L.orc_set_recovery.argtypes = [C.c_void_p, C.c_int32, C.c_double]
            L.orc_combine_scatter.restype = C.c_int32
            L.orc_combine_scatter.argtypes = [u32p, f64p, C.c_int32, u32p, f64p, C.c_int32, C.c_float, C.c_float,
                                              C.c_float, f32p, u32p, f64p, i32p, i32p]
            L.orc_create.restype = C.c_void_p
            L.orc_create.argtypes = [C.c_int64, C.c_int32, C.c_int32, C.c_uint64, C.c_float, C.c_float, C.c_float,
                                     C.c_float]
            L.orc_destroy.restype = None
            L.orc_destroy.argtypes = [C.c_void_p]
            L.orc_set_alpha.restype = None
            L.orc_set_alpha.argtypes = [C.c_void_p, C.c_float]
            for name in ("orc_step_compress",):
                getattr(L, name).restype = None
                getattr(L, name).argtypes = [C.c_void_p, f32p]
            L.orc_step_recover.restype = None
            L.orc_step_recover.argtypes = [C.c_void_p, f32p]
            L.orc_reproject.restype = None
            L.orc_reproject.argtypes = [C.c_void_p, C.c_uint64]
            L.orc_step.restype = None
            L.orc_step.argtypes = [C.c_void_p, f32p, f32p]
            L.orc_get.restype = C.c_int32
            L.orc_get.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_int64]
            L.orc_num_threads.restype = C.c_int32
            L.orc_num_threads.argtypes = []
            _lib = L
    return _lib


def _p(a, ct):
    return a.ctypes.data_as(C.POINTER(ct))


def num_threads():
    return int(lib().orc_num_threads())


def sigma(k):
    """fl32(1/sqrt(k)): the scale of A (standard deviation 1/sqrt(k), Section 3.3)."""
    return np.float32(lib().orc_sigma(int(k)))


def z_block(seed, row0, nrows, col0, ncols):
    """Z(seed, row, col) for a block, as a float32 array [nrows, ncols]; A = sigma(k) * Z."""
    out = np.empty((nrows, ncols), dtype=np.float32)
    lib().orc_z_block(C.c_uint64(seed), row0, nrows, col0, ncols, _p(out, C.c_float))
    return out


def sparsify(g, s):
    g = np.ascontiguousarray(g, dtype=np.float32)
    idx = np.empty(s, dtype=np.uint32)
    val = np.empty(s, dtype=np.float32)
    rc = lib().orc_sparsify(_p(g, C.c_float), g.size, s, _p(idx, C.c_uint32), _p(val, C.c_float))
    if rc != 0:
        raise ValueError("orc_sparsify failed")
    return idx, val


def project(seed, k, idx, val):
    idx = np.ascontiguousarray(idx, dtype=np.uint32)
    val = np.ascontiguousarray(val, dtype=np.float32)
    p = np.empty(k, dtype=np.float64)
    q = np.empty(k, dtype=np.float64)
    lib().orc_project(C.c_uint64(seed), k, _p(idx, C.c_uint32), _p(val, C.c_float), idx.size, _p(p, C.c_double),
                      _p(q, C.c_double))
    return p, q


def adam(M, V, p, q, beta1, beta2, t):
    """In-place update of float32 M, V; returns (Mhat, Vhat) float64."""
    assert M.dtype == np.float32 and V.dtype == np.float32 and M.flags.c_contiguous and V.flags.c_contiguous
    p = np.ascontiguousarray(p, dtype=np.float64)
    q = np.ascontiguousarray(q, dtype=np.float64)
    k = M.size
    Mh = np.empty(k, dtype=np.float64)
    Vh = np.empty(k, dtype=np.float64)
    lib().orc_adam(_p(M, C.c_float), _p(V, C.c_float), _p(p, C.c_double), _p(q, C.c_double), k, beta1, beta2, t,
                   _p(Mh, C.c_double), _p(Vh, C.c_double))
    return Mh, Vh


def omp(seed, d, k, s, y, residual_tol=0.0):
    """Textbook OMP of y against A(seed, k x d).  Returns a dict of per-iteration records.

    residual_tol > 0 ends the iterations once ||r|| <= residual_tol * ||y|| (an opt-in variant; 0 = Algorithm 3's s
    iterations)."""
    y = np.ascontiguousarray(y, dtype=np.float64)
    assert y.size == k
    lam = np.empty(s, dtype=np.uint32)
    x = np.empty(s, dtype=np.float64)
    t1 = np.empty(s, dtype=np.float64)
    t2 = np.empty(s, dtype=np.float64)
    rn = np.empty(s, dtype=np.float64)
    done = lib().orc_omp_tol(C.c_uint64(seed), d, k, s, _p(y, C.c_double), float(residual_tol), _p(lam, C.c_uint32),
                             _p(x, C.c_double), _p(t1, C.c_double), _p(t2, C.c_double), _p(rn, C.c_double))
    return dict(done=int(done), lam=lam, x=x, top1=t1, top2=t2, rnorm=rn)


def select(seed, d, k, R, skip=None):
    """The Select line of Algorithm 3 for a batch of residuals R [n, k] against all d columns of A(seed, k x d).

    skip: optional list of n index sequences, the columns excluded for each residual (its support so far).
    Returns dict(idx [n] int64, best [n], second [n]): argmax column (lowest index on ties) and the two largest scores."""
    R = np.ascontiguousarray(R, dtype=np.float64)
    n = R.shape[0]
    assert R.shape == (n, k)
    counts = np.zeros(n, dtype=np.int32)
    stride = 1
    if skip is not None:
        assert len(skip) == n
        counts = np.array([len(sk) for sk in skip], dtype=np.int32)
        stride = max(1, int(counts.max()))
    flat = np.zeros((n, stride), dtype=np.uint32)
    if skip is not None:
        for i, sk in enumerate(skip):
            flat[i, :len(sk)] = np.asarray(sk, dtype=np.uint32)
    idx = np.empty(n, dtype=np.int64)
    best = np.empty(n, dtype=np.float64)
    second = np.empty(n, dtype=np.float64)
    lib().orc_select(C.c_uint64(seed), int(d), int(k), n, _p(R, C.c_double), _p(flat, C.c_uint32), _p(counts, C.c_int32),
                     stride, _p(idx, C.c_int64), _p(best, C.c_double), _p(second, C.c_double))
    return dict(idx=idx, best=best, second=second)


def least_squares(seed, k, lam, y):
    """argmin_x ||y - A_lam x||_2 for the columns lam of A(seed, k x .): the last step of an OMP iteration on its own."""
    lam = np.ascontiguousarray(lam, dtype=np.uint32)
    y = np.ascontiguousarray(y, dtype=np.float64)
    assert y.size == k
    x = np.zeros(lam.size, dtype=np.float64)
    rc = lib().orc_least_squares(C.c_uint64(seed), k, _p(lam, C.c_uint32), lam.size, _p(y, C.c_double), _p(x, C.c_double))
    if rc != 0:
        raise ValueError("dependent columns")
    return x


def combine_scatter(lamM, xM, lamV, xV, alpha, eps, lr, W):
    """Applies Eq. (8) + Eq. (3) to float32 W in place; returns (upd_idx, upd_val, mismatch, negv)."""
    lamM = np.ascontiguousarray(lamM, dtype=np.uint32)
    lamV = np.ascontiguousarray(lamV, dtype=np.uint32)
    xM = np.ascontiguousarray(xM, dtype=np.float64)
    xV = np.ascontiguousarray(xV, dtype=np.float64)
    assert W.dtype == np.float32 and W.flags.c_contiguous
    cap = max(lamM.size, 1)
    ui = np.empty(cap, dtype=np.uint32)
    uv = np.empty(cap, dtype=np.float64)
    mis = C.c_int32(0)
    neg = C.c_int32(0)
    n = lib().orc_combine_scatter(_p(lamM, C.c_uint32), _p(xM, C.c_double), lamM.size, _p(lamV, C.c_uint32),
                                  _p(xV, C.c_double), lamV.size, alpha, eps, lr, _p(W, C.c_float),
                                  _p(ui, C.c_uint32), _p(uv, C.c_double), C.byref(mis), C.byref(neg))
    return ui[:n].copy(), uv[:n].copy(), mis.value, neg.value


_GET = dict(t=(0, np.int64, None), M=(1, np.float32, "k"), V=(2, np.float32, "k"), p=(3, np.float64, "k"),
            q=(4, np.float64, "k"), sel_idx=(5, np.uint32, "s"), sel_val=(6, np.float32, "s"),
            lamM=(7, np.uint32, "s"), lamV=(8, np.uint32, "s"), xM=(9, np.float64, "s"), xV=(10, np.float64, "s"),
            top1M=(11, np.float64, "s"), top2M=(12, np.float64, "s"), top1V=(13, np.float64, "s"),
            top2V=(14, np.float64, "s"), upd_idx=(15, np.uint32, "s"), upd_val=(16, np.float64, "s"),
            n_upd=(17, np.int32, None), mismatch=(18, np.int32, None), negv=(19, np.int32, None),
            doneM=(20, np.int32, None), doneV=(21, np.int32, None), Mhat=(22, np.float64, "k"),
            Vhat=(23, np.float64, "k"), rnormM=(24, np.float64, "s"), rnormV=(25, np.float64, "s"))


class Oracle:
    """Stateful oracle with the same life cycle as the product's sgc_create / sgc_step / sgc_destroy."""

    def __init__(self, d, k, s, seed, lr, beta1, beta2, eps, alpha=1.0):
        self.d, self.k, self.s = int(d), int(k), int(s)
        self._h = lib().orc_create(self.d, self.k, self.s, C.c_uint64(seed), lr, beta1, beta2, eps)
        if not self._h:
            raise ValueError("orc_create rejected the arguments")
        if alpha != 1.0:
            lib().orc_set_alpha(self._h, alpha)

    def close(self):
        if self._h:
            lib().orc_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _g(self, grad):
        assert grad.dtype == np.float32 and grad.flags.c_contiguous and grad.size == self.d
        return _p(grad, C.c_float)

    def step_compress(self, grad):
        lib().orc_step_compress(self._h, self._g(grad))

    def step_recover(self, weight):
        assert weight.dtype == np.float32 and weight.flags.c_contiguous and weight.size == self.d
        lib().orc_step_recover(self._h, _p(weight, C.c_float))

    def step(self, grad, weight):
        self.step_compress(grad)
        self.step_recover(weight)

    def set_recovery(self, shared_support, residual_tol=0.0):
        """Opt-in variant: one support (that of OMP_A(M^)) for both moments, and / or an early stop on ||r||."""
        lib().orc_set_recovery(self._h, 1 if shared_support else 0, float(residual_tol))

    def reproject(self, new_seed):
        """SGCA (Algorithm 4): M <- A' OMP_A(M), V <- A' OMP_A(V), A <- A' with A' named by new_seed."""
        lib().orc_reproject(self._h, C.c_uint64(new_seed))

    def get(self, name):
        what, dt, dim = _GET[name]
        n = 1 if dim is None else getattr(self, dim)
        out = np.empty(n, dtype=dt)
        rc = lib().orc_get(self._h, what, out.ctypes.data_as(C.c_void_p), out.nbytes)
        if rc != 0:
            raise RuntimeError("orc_get(%s) failed: %d" % (name, rc))
        return out[0] if dim is None else out


def cesgc_step(chunks, B, G, W):
    """One CESGC step (Section 4.4, "Compute Efficient SGC") written out from its definition, W <- W - eta B^T SGC(B G).

    chunks: the c chunk oracles (Oracle objects of length r * n / c each, same seed: MESGC on the projected gradient);
    B: float32 [r, m]; G: float32 [m, n]; W: float32 [m, n], updated in place.  P = B G is formed in fp64 and rounded
    to float32 (the gradient the SGC core is given); every chunk steps on its slice of P with zero "weights", which
    leaves -eta N there; the result goes back through B^T in fp64.  Returns (P, U) with U = -eta N as float32 [r, n]."""
    r, m = B.shape
    n = G.shape[1]
    assert G.shape == (m, n) and W.shape == (m, n) and W.dtype == np.float32
    P = (B.astype(np.float64) @ G.astype(np.float64)).astype(np.float32)
    U = np.zeros(r * n, dtype=np.float32)
    dc = r * n // len(chunks)
    flat = P.reshape(-1)
    for i, ch in enumerate(chunks):
        ch.step(np.ascontiguousarray(flat[i * dc:(i + 1) * dc]), U[i * dc:(i + 1) * dc])
    U2 = U.reshape(r, n)
    W[...] = (W.astype(np.float64) + B.astype(np.float64).T @ U2.astype(np.float64)).astype(np.float32)
    return P, U2
