"""ctypes front end of the SubGen oracle (``subgen_oracle.c``).

TEST INFRASTRUCTURE ONLY: a slow CPU statement of Algorithm 1 of the SubGen
paper (UpdateSoftmaxNormalizer, UpdateMatrixProduct, QueryStreamAttn) with the
sliding window of its Section 3.2. Tests, the smoke check and the CPU-baseline
leg of the benchmark may import it; the CUDA library and its Python binding
never do, and it imports nothing of theirs.

All arithmetic lives in the C file; this module only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "subgen_oracle.c")
_LIB = os.path.join(_HERE, "libsubgen_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            subprocess.check_call(
                ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
                 "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        path = build()
        with _lock:
            if _lib is None:
                L = C.CDLL(path)
                fp = C.POINTER(C.c_float)
                dp = C.POINTER(C.c_double)
                ip = C.POINTER(C.c_int)
                up = C.POINTER(C.c_uint64)
                vp = C.c_void_p
                L.oracle_philox4x32_10.argtypes = [C.POINTER(C.c_uint32)] * 3
                L.oracle_create.restype = vp
                L.oracle_create.argtypes = [C.c_int, C.c_float, C.c_int, C.c_int, C.c_int,
                                            C.c_uint64, C.c_uint32, C.c_int]
                L.oracle_destroy.argtypes = [vp]
                L.oracle_push.argtypes = [vp, fp, fp]
                L.oracle_push_many.argtypes = [vp, fp, fp, C.c_int]
                L.oracle_query.argtypes = [vp, fp, dp]
                L.oracle_query_parts.argtypes = [vp, fp, dp, dp, dp, dp]
                L.oracle_step.argtypes = [vp, fp, fp, fp, dp]
                L.oracle_exact_attention.argtypes = [fp, fp, C.c_int, C.c_int, fp, dp]
                for name in ("oracle_n", "oracle_inserted", "oracle_m", "oracle_overflow_at"):
                    getattr(L, name).argtypes = [vp]
                    getattr(L, name).restype = C.c_int
                L.oracle_set_bounded.argtypes = [vp, C.c_int]
                L.oracle_level.argtypes = [vp]
                L.oracle_level.restype = C.c_int
                for name in ("oracle_mu", "oracle_delta2_fx", "oracle_thr2_fx"):
                    getattr(L, name).argtypes = [vp]
                    getattr(L, name).restype = C.c_uint64
                for name in ("oracle_counts", "oracle_centre_tok", "oracle_slot_tok", "oracle_m_tok",
                             "oracle_assign", "oracle_ins_near"):
                    getattr(L, name).argtypes = [vp]
                    getattr(L, name).restype = ip
                for name in ("oracle_w", "oracle_ins_d2"):
                    getattr(L, name).argtypes = [vp]
                    getattr(L, name).restype = up
                L.oracle_kcenter.argtypes = [fp, C.c_int, C.c_int, C.c_int, ip, up]
                L.oracle_kcenter.restype = C.c_int
                L.oracle_dist2_fx.argtypes = [fp, fp, C.c_int]
                L.oracle_dist2_fx.restype = C.c_uint64
                L.oracle_norm2_fx.argtypes = [fp, C.c_int]
                L.oracle_norm2_fx.restype = C.c_uint64
                _lib = L
    return _lib


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def _fp(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_float))


def philox4x32_10(counter, key):
    """Philox4x32-10 block: 4 counter words, 2 key words -> 4 output words."""
    c = (C.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in counter])
    k = (C.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    o = (C.c_uint32 * 4)()
    lib().oracle_philox4x32_10(c, k, o)
    return [int(x) for x in o]


def exact_attention(K, V, q) -> np.ndarray:
    """Eq. 1: softmax(K q)^T V, fp64 accumulation over binary32 inputs."""
    K = _f32(K); V = _f32(V); q = _f32(q)
    n, d = K.shape
    out = np.zeros(d, dtype=np.float64)
    lib().oracle_exact_attention(_fp(K), _fp(V), n, d, _fp(q), out.ctypes.data_as(C.POINTER(C.c_double)))
    return out


def dist2_fx(x, k) -> int:
    x = _f32(x); k = _f32(k)
    return int(lib().oracle_dist2_fx(_fp(x), _fp(k), x.shape[0]))


def norm2_fx(v) -> int:
    v = _f32(v)
    return int(lib().oracle_norm2_fx(_fp(v), v.shape[0]))


def kcenter(K_old, k):
    """Greedy k-center over the rows of K_old (first centre = row 0, farthest-point traversal, fixed-point
    distances, ties to the lowest index). Returns (centres in selection order, covering radius^2 in fixed point)."""
    K_old = _f32(K_old)
    n, d = K_old.shape
    out = np.zeros(max(min(k, n), 1), dtype=np.int32)
    rad = C.c_uint64(0)
    kk = lib().oracle_kcenter(_fp(K_old), n, d, int(k), out.ctypes.data_as(C.POINTER(C.c_int)), C.byref(rad))
    return out[:kk].copy(), int(rad.value)


def kcenter_window_attention(K, V, q, k, r):
    """Section 3.2 variant: exact attention (Eq. 1) over k greedy centres of the n - r oldest tokens plus the r most
    recent tokens. Returns (out, kept token indices: centres in selection order, then the window)."""
    K = _f32(K); V = _f32(V)
    n = K.shape[0]
    n_old = max(0, n - r)
    cent, _ = kcenter(K[:n_old], k) if n_old else (np.zeros(0, np.int32), 0)
    keep = np.concatenate([cent.astype(np.int64), np.arange(n_old, n)])
    return exact_attention(K[keep], V[keep], q), keep


class OracleUnit:
    """One stream = one (sequence, KV head) unit of the SubGen data structure."""

    def __init__(self, d, delta, t, s, window, seed=0, unit_id=0, m_max=1 << 16, bounded=False):
        """bounded=True: m_max is a budget; when it is exhausted the threshold doubles and clusters merge
        (the doubling_sweep of the C file) instead of the stream failing."""
        self.d, self.t, self.s, self.window, self.m_max = int(d), int(t), int(s), int(window), int(m_max)
        self._L = lib()
        self._h = self._L.oracle_create(self.d, float(np.float32(delta)), self.t, self.s, self.window,
                                        int(seed) & (2 ** 64 - 1), int(unit_id), self.m_max)
        if not self._h:
            raise ValueError("oracle_create rejected its arguments")
        if bounded:
            self._L.oracle_set_bounded(self._h, 1)

    def close(self):
        if getattr(self, "_h", None):
            self._L.oracle_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- stream ---------------------------------------------------------------
    def push(self, k, v):
        k = _f32(k); v = _f32(v)
        if self._L.oracle_push(self._h, _fp(k), _fp(v)):
            raise OverflowError("cluster capacity m_max exceeded at token %d" % self.overflow_at)

    def push_many(self, K, V):
        K = _f32(K); V = _f32(V)
        assert K.shape == V.shape and K.ndim == 2 and K.shape[1] == self.d
        if K.shape[0] and self._L.oracle_push_many(self._h, _fp(K), _fp(V), K.shape[0]):
            raise OverflowError("cluster capacity m_max exceeded at token %d" % self.overflow_at)

    def query(self, q) -> np.ndarray:
        q = _f32(q)
        out = np.zeros(self.d, dtype=np.float64)
        self._L.oracle_query(self._h, _fp(q), out.ctypes.data_as(C.POINTER(C.c_double)))
        return out

    def query_parts(self, q):
        """Returns (out, z, tau, shift): z and tau are scaled by exp(-shift)."""
        q = _f32(q)
        out = np.zeros(self.d, dtype=np.float64)
        z = np.zeros(self.d, dtype=np.float64)
        tau = C.c_double(0.0)
        shift = C.c_double(0.0)
        dp = C.POINTER(C.c_double)
        self._L.oracle_query_parts(self._h, _fp(q), out.ctypes.data_as(dp), z.ctypes.data_as(dp),
                                   C.byref(tau), C.byref(shift))
        return out, z, tau.value, shift.value

    def step(self, q, k, v) -> np.ndarray:
        self.push(k, v)
        return self.query(q)

    # -- state ----------------------------------------------------------------
    def _ints(self, fn, n):
        p = fn(self._h)
        return np.ctypeslib.as_array(p, shape=(n,)).copy() if n else np.zeros(0, dtype=np.int32)

    def _u64s(self, fn, n):
        p = fn(self._h)
        return np.ctypeslib.as_array(p, shape=(n,)).copy() if n else np.zeros(0, dtype=np.uint64)

    @property
    def n(self): return self._L.oracle_n(self._h)
    @property
    def inserted(self): return self._L.oracle_inserted(self._h)
    @property
    def m(self): return self._L.oracle_m(self._h)
    @property
    def mu(self): return int(self._L.oracle_mu(self._h))
    @property
    def delta2_fx(self): return int(self._L.oracle_delta2_fx(self._h))
    @property
    def thr2_fx(self): return int(self._L.oracle_thr2_fx(self._h))
    @property
    def level(self): return self._L.oracle_level(self._h)
    @property
    def overflow_at(self): return self._L.oracle_overflow_at(self._h)
    @property
    def counts(self): return self._ints(self._L.oracle_counts, self.m)
    @property
    def centre_tok(self): return self._ints(self._L.oracle_centre_tok, self.m)
    @property
    def slot_tok(self): return self._ints(self._L.oracle_slot_tok, self.m * self.t).reshape(self.m, self.t)
    @property
    def m_tok(self): return self._ints(self._L.oracle_m_tok, self.s)
    @property
    def assign(self): return self._ints(self._L.oracle_assign, self.n)
    @property
    def w(self): return self._u64s(self._L.oracle_w, self.n)
    @property
    def ins_d2(self): return self._u64s(self._L.oracle_ins_d2, self.n)
    @property
    def ins_near(self): return self._ints(self._L.oracle_ins_near, self.n)
