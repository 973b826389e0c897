"""Thin ctypes binding of libsubgen.so (declared in include/subgen.h).

Argument marshalling only: every step of the path runs in the library's CUDA kernels. torch is used
for device memory and streams. There is no CPU path: loading fails loudly if the shared library is
missing, and every call fails if no CUDA device is usable.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsubgen.so")

DTYPE_FP32, DTYPE_BF16 = 0, 1
ST_CAPACITY, ST_RANGE = 1, 2
STEP_MODES = {"auto": 0, "fused": 1, "split": 2}

EXPORTS = [
    "subgen_workspace_bytes", "subgen_create", "subgen_create_ex", "subgen_destroy", "subgen_prefill",
    "subgen_prefill_varlen", "subgen_step", "subgen_step_host", "subgen_status", "subgen_export_state",
    "subgen_export_rows", "subgen_cache_stats", "subgen_profile_enable", "subgen_profile_read", "subgen_profile_prefill_read",
    "subgen_query", "subgen_launch_count", "subgen_step_kernels", "subgen_last_error", "subgen_checkpoint_bytes", "subgen_checkpoint_save", "subgen_checkpoint_load", "subgen_grow", "subgen_exact_create", "subgen_exact_destroy",
    "subgen_exact_append", "subgen_exact_append_varlen", "subgen_exact_step", "subgen_exact_bytes",
    "subgen_exact_launch_count", "subgen_exact_attention_noalloc",
    "subgen_exact_kcenter_compress", "subgen_exact_kcenter_counters", "subgen_exact_export_tokens",
]


class SubgenConfig(C.Structure):
    _fields_ = [("B", C.c_int), ("H", C.c_int), ("Hkv", C.c_int), ("d", C.c_int), ("delta", C.c_float),
                ("t", C.c_int), ("s", C.c_int), ("window", C.c_int), ("seed", C.c_uint64), ("dtype", C.c_int),
                ("m_max", C.c_int), ("splits", C.c_int), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
                ("stream", C.c_void_p), ("nq_max", C.c_int), ("bounded", C.c_int), ("step_mode", C.c_int),
                ("unit_stride", C.c_int), ("unit_offset", C.c_int)]


class StateView(C.Structure):
    _fields_ = [("n", C.c_int), ("inserted", C.c_int), ("m", C.c_int), ("status", C.c_int), ("mu", C.c_uint64),
                ("last_cluster", C.c_int), ("last_opened", C.c_int), ("last_d2", C.c_uint64),
                ("counts", C.c_void_p), ("centre_tok", C.c_void_p), ("slot_tok", C.c_void_p),
                ("m_tok", C.c_void_p), ("m_w", C.c_void_p), ("threshold2", C.c_uint64), ("doublings", C.c_int)]


class Stats(C.Structure):
    _fields_ = [(k, C.c_uint64) for k in ("units", "clusters", "singleton_clusters", "m_filled", "window_rows",
                                           "tokens", "prefill_pairs", "insert_bytes", "query_bytes", "cluster_bytes", "value_bytes",
                                           "distinct_sample_rows")]


_lib = None


def load():
    """Load libsubgen.so; raises if it has not been built (python -m paper_2402_06082_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("libsubgen.so is missing: build it with `python paper_2402_06082_b200/build.py`; "
                           "there is no fallback path")
    L = C.CDLL(LIB_PATH)
    vp, ip = C.c_void_p, C.POINTER(C.c_int)
    L.subgen_workspace_bytes.restype = C.c_size_t
    L.subgen_workspace_bytes.argtypes = [C.POINTER(SubgenConfig)]
    L.subgen_create.restype = vp
    L.subgen_create.argtypes = [C.c_int, C.c_int, C.c_int, C.c_float, C.c_int, C.c_int, C.c_int, C.c_uint64]
    L.subgen_create_ex.restype = vp
    L.subgen_create_ex.argtypes = [C.POINTER(SubgenConfig)]
    L.subgen_destroy.argtypes = [vp]
    L.subgen_destroy.restype = None
    L.subgen_prefill.argtypes = [vp, vp, vp, C.c_int]
    L.subgen_prefill_varlen.argtypes = [vp, vp, vp, ip]
    L.subgen_step.argtypes = [vp, vp, vp, vp, vp]
    L.subgen_step_host.argtypes = [vp, vp, vp, vp, vp]
    L.subgen_status.argtypes = [vp]
    L.subgen_export_state.argtypes = [vp, C.c_int, C.c_int, C.POINTER(StateView)]
    L.subgen_export_rows.argtypes = [vp, C.c_int, C.c_int, C.c_int, vp, C.c_size_t]
    L.subgen_cache_stats.argtypes = [vp, C.POINTER(Stats)]
    L.subgen_profile_enable.argtypes = [vp, C.c_int]
    L.subgen_profile_read.argtypes = [vp, C.POINTER(C.c_double), ip]
    L.subgen_profile_prefill_read.argtypes = [vp, C.POINTER(C.c_double)]
    L.subgen_launch_count.argtypes = [vp]
    L.subgen_step_kernels.argtypes = [vp]
    L.subgen_query.argtypes = [vp, vp, C.c_int, vp]
    L.subgen_checkpoint_bytes.argtypes = [vp, C.POINTER(C.c_size_t)]
    L.subgen_checkpoint_save.argtypes = [vp, vp, C.c_size_t, C.POINTER(C.c_size_t)]
    L.subgen_checkpoint_load.argtypes = [vp, vp, C.c_size_t]
    L.subgen_grow.argtypes = [vp, C.c_int, vp, C.c_size_t]
    L.subgen_launch_count.restype = C.c_uint64
    L.subgen_last_error.restype = C.c_char_p
    L.subgen_exact_create.restype = vp
    L.subgen_exact_create.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, vp]
    L.subgen_exact_destroy.argtypes = [vp]
    L.subgen_exact_destroy.restype = None
    L.subgen_exact_append.argtypes = [vp, vp, vp, C.c_int]
    L.subgen_exact_append_varlen.argtypes = [vp, vp, vp, ip]
    L.subgen_exact_step.argtypes = [vp, vp, vp, vp, vp]
    L.subgen_exact_bytes.argtypes = [vp, C.POINTER(C.c_uint64)]
    L.subgen_exact_launch_count.argtypes = [vp]
    L.subgen_exact_launch_count.restype = C.c_uint64
    L.subgen_exact_kcenter_compress.argtypes = [vp, C.c_int, C.c_int]
    L.subgen_exact_kcenter_counters.argtypes = [vp, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
    L.subgen_exact_export_tokens.argtypes = [vp, C.c_int, C.c_int, ip, ip]
    L.subgen_exact_attention_noalloc.argtypes = [vp, vp, vp, vp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, vp]
    _lib = L
    return L


class SubgenError(RuntimeError):
    pass


def _check(rc: int):
    if rc < 0:
        raise SubgenError("subgen error %d: %s" % (rc, load().subgen_last_error().decode()))
    return rc


def _dtype_code(dt: torch.dtype) -> int:
    if dt == torch.float32:
        return DTYPE_FP32
    if dt == torch.bfloat16:
        return DTYPE_BF16
    raise ValueError("dtype must be torch.float32 or torch.bfloat16")


def _dev(x: torch.Tensor, dt: torch.dtype, shape: Sequence[int], name: str) -> int:
    if not (x.is_cuda and x.is_contiguous() and x.dtype == dt and tuple(x.shape) == tuple(shape)):
        raise ValueError("%s must be a contiguous CUDA %s tensor of shape %s (got %s %s)" %
                         (name, dt, tuple(shape), x.dtype, tuple(x.shape)))
    return x.data_ptr()


class SubGen:
    """One library handle: the SubGen caches of B sequences x Hkv KV heads on the current CUDA device."""

    def __init__(self, B, H, d, delta, t, s, window, seed=0, *, Hkv=None, dtype=torch.bfloat16, m_max=0, splits=0,
                 stream: Optional[torch.cuda.Stream] = None, bounded: bool = False, nq_max: int = 1,
                 step_mode: str = "auto", unit_stride: int = 0, unit_offset: int = 0):
        self._L = load()
        self._h = None
        if not torch.cuda.is_available():
            raise SubgenError("no CUDA device: this library has no CPU path")
        self.bounded = bool(bounded)
        self.B, self.H, self.Hkv, self.d = int(B), int(H), int(Hkv or H), int(d)
        self.t, self.s, self.window, self.dtype = int(t), int(s), int(window), dtype
        self.stream = stream or torch.cuda.current_stream()
        cfg = SubgenConfig(self.B, self.H, self.Hkv, self.d, float(delta), self.t, self.s, self.window, int(seed),
                           _dtype_code(dtype), int(m_max), int(splits), None, 0, self.stream.cuda_stream, int(nq_max), int(bool(bounded)),
                           STEP_MODES[step_mode], int(unit_stride), int(unit_offset))
        nbytes = self._L.subgen_workspace_bytes(C.byref(cfg))
        if nbytes == 0:
            raise SubgenError(self._L.subgen_last_error().decode())
        self._cfg = cfg
        self.m_max = int(m_max) if m_max else 8192
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")   # torch owns the memory
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        cfg.workspace, cfg.workspace_bytes = base, nbytes
        self.workspace_bytes = nbytes
        self._h = self._L.subgen_create_ex(C.byref(cfg))
        if not self._h:
            raise SubgenError(self._L.subgen_last_error().decode())

    def close(self):
        if self._h:
            self._L.subgen_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- stream ---------------------------------------------------------------------------------
    def prefill(self, K: torch.Tensor, V: torch.Tensor):
        n = K.shape[2]
        shp = (self.B, self.Hkv, n, self.d)
        _check(self._L.subgen_prefill(self._h, _dev(K, self.dtype, shp, "K"), _dev(V, self.dtype, shp, "V"), n))

    def prefill_varlen(self, K: torch.Tensor, V: torch.Tensor, cu_seqlens: Sequence[int]):
        cu = (C.c_int * (self.B + 1))(*[int(x) for x in cu_seqlens])
        shp = (self.Hkv, int(cu_seqlens[-1]), self.d)
        _check(self._L.subgen_prefill_varlen(self._h, _dev(K, self.dtype, shp, "K"), _dev(V, self.dtype, shp, "V"), cu))

    def step(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: Optional[torch.Tensor] = None):
        qs, ks = (self.B, self.H, self.d), (self.B, self.Hkv, self.d)
        if out is None:
            out = torch.empty(qs, dtype=self.dtype, device="cuda")
        _check(self._L.subgen_step(self._h, _dev(q, self.dtype, qs, "q"), _dev(k, self.dtype, ks, "k"),
                                   _dev(v, self.dtype, ks, "v"), _dev(out, self.dtype, qs, "out")))
        return out

    def query(self, q: torch.Tensor, out: Optional[torch.Tensor] = None):
        """Read-only QueryStreamAttn for nq queries per head: q [B, H, nq, d] -> out [B, H, nq, d]."""
        nq = int(q.shape[2])
        qs = (self.B, self.H, nq, self.d)
        if out is None:
            out = torch.empty(qs, dtype=self.dtype, device="cuda")
        _check(self._L.subgen_query(self._h, _dev(q, self.dtype, qs, "q"), nq, _dev(out, self.dtype, qs, "out")))
        return out

    def step_host(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: torch.Tensor):
        """q, k, v, out are HOST tensors (pinned for asynchronous copies); returns when out is filled."""
        for x in (q, k, v, out):
            if x.is_cuda or not x.is_contiguous() or x.dtype != self.dtype:
                raise ValueError("step_host takes contiguous host tensors of the handle's dtype")
        _check(self._L.subgen_step_host(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr()))
        return out

    def status(self) -> int:
        return _check(self._L.subgen_status(self._h))

    # ---- inspection -----------------------------------------------------------------------------
    def export_state(self, seq: int, kvhead: int) -> dict:
        counts = np.zeros(self.m_max, np.int32)
        ctok = np.zeros(self.m_max, np.int32)
        stok = np.zeros(self.m_max * self.t, np.int32)
        mtok = np.zeros(self.s, np.int32)
        mw = np.zeros(self.s, np.uint64)
        v = StateView()
        v.counts, v.centre_tok, v.slot_tok = counts.ctypes.data, ctok.ctypes.data, stok.ctypes.data
        v.m_tok, v.m_w = mtok.ctypes.data, mw.ctypes.data
        _check(self._L.subgen_export_state(self._h, seq, kvhead, C.byref(v)))
        m = v.m
        return dict(n=v.n, inserted=v.inserted, m=m, status=v.status, mu=int(v.mu), last_cluster=v.last_cluster,
                    last_opened=v.last_opened, last_d2=int(v.last_d2), counts=counts[:m].copy(),
                    centre_tok=ctok[:m].copy(), slot_tok=stok.reshape(self.m_max, self.t)[:m].copy(),
                    m_tok=mtok, m_w=mw, threshold2=int(v.threshold2), doublings=v.doublings)

    def export_rows(self, seq: int, kvhead: int, which: int) -> torch.Tensor:
        rows = {0: self.m_max, 1: self.m_max * self.t, 2: self.s, 3: self.s, 4: self.window, 5: self.window}[which]
        buf = torch.empty((rows, self.d), dtype=self.dtype)
        _check(self._L.subgen_export_rows(self._h, seq, kvhead, which, buf.data_ptr(), buf.numel() * buf.element_size()))
        return buf

    def cache_stats(self) -> dict:
        s = Stats()
        _check(self._L.subgen_cache_stats(self._h, C.byref(s)))
        return {k: int(getattr(s, k)) for k, _ in Stats._fields_}

    def profile_enable(self, on: bool = True):
        _check(self._L.subgen_profile_enable(self._h, int(on)))

    def profile_read(self):
        """(insert_ms, cluster_scan_ms, value_scan_ms, steps) accumulated since the last read."""
        ms, n = (C.c_double * 3)(), C.c_int()
        _check(self._L.subgen_profile_read(self._h, ms, C.byref(n)))
        return ms[0], ms[1], ms[2], n.value

    def profile_prefill_read(self):
        """(value_phase_ms, score_ms, resolve_ms) of the last chunked prefill made with profiling enabled."""
        ms = (C.c_double * 3)()
        _check(self._L.subgen_profile_prefill_read(self._h, ms))
        return ms[0], ms[1], ms[2]

    @property
    def launch_count(self) -> int:
        return int(self._L.subgen_launch_count(self._h))

    @property
    def step_kernels(self) -> int:
        """Kernels one step launches: 1 (fused step), 2 (fp32) or 3."""
        return _check(self._L.subgen_step_kernels(self._h))

    def checkpoint_save(self) -> torch.Tensor:
        """The state between two calls as one pinned uint8 host tensor (see subgen_checkpoint_save)."""
        n = C.c_size_t()
        _check(self._L.subgen_checkpoint_bytes(self._h, C.byref(n)))
        blob = torch.empty(n.value, dtype=torch.uint8, pin_memory=True)
        w = C.c_size_t()
        _check(self._L.subgen_checkpoint_save(self._h, blob.data_ptr(), n.value, C.byref(w)))
        return blob[: w.value]

    def checkpoint_load(self, blob: torch.Tensor):
        """Replace this handle's state by a saved one; the configuration must match, m_max may be larger."""
        if blob.dtype != torch.uint8 or blob.device.type != "cpu" or not blob.is_contiguous():
            raise ValueError("blob must be a contiguous uint8 host tensor")
        _check(self._L.subgen_checkpoint_load(self._h, blob.data_ptr(), blob.numel()))

    def grow(self, m_max: int):
        """Re-lay the state out for a larger cluster capacity per unit (see subgen_grow); the stream continues unchanged."""
        cfg = SubgenConfig.from_buffer_copy(self._cfg)
        cfg.m_max = int(m_max)
        cfg.workspace, cfg.workspace_bytes = None, 0
        nbytes = self._L.subgen_workspace_bytes(C.byref(cfg))
        if nbytes == 0:
            raise SubgenError(self._L.subgen_last_error().decode())
        ws = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
        base = (ws.data_ptr() + 255) // 256 * 256
        _check(self._L.subgen_grow(self._h, int(m_max), base, nbytes))
        self.workspace, self.workspace_bytes = ws, nbytes            # the old tensor is released here
        self._cfg.m_max = int(m_max)
        self.m_max = int(m_max)


class ExactAttention:
    """Exact dense decode attention over a full KV cache (Eq. 1), the comparison point."""

    def __init__(self, B, H, d, n_max, *, Hkv=None, dtype=torch.bfloat16, stream: Optional[torch.cuda.Stream] = None):
        self._L = load()
        self._h = None
        if not torch.cuda.is_available():
            raise SubgenError("no CUDA device: this library has no CPU path")
        self.B, self.H, self.Hkv, self.d, self.n_max, self.dtype = int(B), int(H), int(Hkv or H), int(d), int(n_max), dtype
        self.stream = stream or torch.cuda.current_stream()
        self._h = self._L.subgen_exact_create(self.B, self.H, self.Hkv, self.d, self.n_max, _dtype_code(dtype),
                                              self.stream.cuda_stream)
        if not self._h:
            raise SubgenError(self._L.subgen_last_error().decode())

    def close(self):
        if self._h:
            self._L.subgen_exact_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def append(self, K, V):
        n = K.shape[2]
        shp = (self.B, self.Hkv, n, self.d)
        _check(self._L.subgen_exact_append(self._h, _dev(K, self.dtype, shp, "K"), _dev(V, self.dtype, shp, "V"), n))

    def append_varlen(self, K, V, cu_seqlens):
        cu = (C.c_int * (self.B + 1))(*[int(x) for x in cu_seqlens])
        shp = (self.Hkv, int(cu_seqlens[-1]), self.d)
        _check(self._L.subgen_exact_append_varlen(self._h, _dev(K, self.dtype, shp, "K"), _dev(V, self.dtype, shp, "V"), cu))

    def step(self, q, k, v, out=None):
        qs, ks = (self.B, self.H, self.d), (self.B, self.Hkv, self.d)
        if out is None:
            out = torch.empty(qs, dtype=self.dtype, device="cuda")
        _check(self._L.subgen_exact_step(self._h, _dev(q, self.dtype, qs, "q"), _dev(k, self.dtype, ks, "k"),
                                         _dev(v, self.dtype, ks, "v"), _dev(out, self.dtype, qs, "out")))
        return out

    def kcenter_compress(self, k: int, r: int):
        """Keep the r most recent tokens and k greedy k-center centres of the older ones (Section 3.2 variant)."""
        _check(self._L.subgen_exact_kcenter_compress(self._h, int(k), int(r)))

    def kcenter_counters(self):
        """(tokens looked at, full key rows read) of the last compression, summed over units and passes."""
        a, b = C.c_uint64(), C.c_uint64()
        _check(self._L.subgen_exact_kcenter_counters(self._h, C.byref(a), C.byref(b)))
        return int(a.value), int(b.value)

    def export_tokens(self, seq: int, kvhead: int) -> np.ndarray:
        n = C.c_int()
        buf = np.zeros(self.n_max, np.int32)
        _check(self._L.subgen_exact_export_tokens(self._h, seq, kvhead, C.byref(n), buf.ctypes.data_as(C.POINTER(C.c_int))))
        return buf[: n.value].copy()

    def bytes_per_step(self) -> int:
        b = C.c_uint64()
        _check(self._L.subgen_exact_bytes(self._h, C.byref(b)))
        return int(b.value)

    @property
    def launch_count(self) -> int:
        return int(self._L.subgen_exact_launch_count(self._h))


NOALLOC_SCRATCH_BYTES = 4 << 20


def exact_attention_noalloc(q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, out: torch.Tensor,
                            stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """out = softmax(K q)^T V per head without any device allocation by the library.

    For callers that may not call cudaMalloc (a plugin inside a process whose allocator owns all device
    memory, or request-path code that cannot take an allocation's synchronisation): the split partials
    live in a fixed array inside the library image (NOALLOC_SCRATCH_BYTES per GPU, shared by all calls,
    so calls that can overlap on the GPU must be ordered). q, out: CUDA [B, H, d]; K, V: CUDA [B, Hkv, n, d].
    The caller supplies `out`; this wrapper creates no tensor.
    """
    B, H, d = q.shape
    Hkv, n = K.shape[1], K.shape[2]
    dt = q.dtype
    st = stream or torch.cuda.current_stream()
    _check(load().subgen_exact_attention_noalloc(
        _dev(q, dt, (B, H, d), "q"), _dev(K, dt, (B, Hkv, n, d), "K"), _dev(V, dt, (B, Hkv, n, d), "V"),
        _dev(out, dt, (B, H, d), "out"), B, H, Hkv, d, n, _dtype_code(dt), st.cuda_stream))
    return out
