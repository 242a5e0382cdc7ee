"""ctypes access to the CPU oracle (oracle/triaccel_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, the smoke check and the benchmark's
CPU-baseline leg.  It imports nothing from the CUDA package and the CUDA package
imports nothing from here.  Arrays are numpy, on the host.
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

FP16, BF16, FP32 = 0, 1, 2


class Segment(C.Structure):
    _fields_ = [("offset", C.c_uint64), ("length", C.c_uint64)]


class HParams(C.Structure):
    _fields_ = [("beta", C.c_float), ("tau_low", C.c_float), ("tau_high", C.c_float),
                ("tau_curv", C.c_float), ("alpha", C.c_float), ("eta0", C.c_float),
                ("topk_ppm", C.c_uint32), ("num_probes", C.c_uint32), ("t_ctrl", C.c_uint32),
                ("grad_dtype", C.c_uint32), ("momentum", C.c_float), ("weight_decay", C.c_float)]


class Layer(C.Structure):
    _fields_ = [("grad_mean", C.c_double), ("grad_var", C.c_double), ("topk_mass", C.c_double),
                ("ema_mean", C.c_float), ("ema_var", C.c_float), ("lambda_max", C.c_float),
                ("topk_threshold", C.c_float), ("eta_scale", C.c_float), ("code", C.c_uint32),
                ("k", C.c_uint64), ("near_threshold", C.c_uint32), ("pad", C.c_uint32)]


class Status(C.Structure):
    _fields_ = [("step", C.c_uint64), ("nonfinite_count", C.c_uint64), ("skipped", C.c_uint32),
                ("near_threshold_count", C.c_uint32)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        path = _build.build()
        L = C.CDLL(path)
        L.orc_create.restype = C.c_void_p
        L.orc_create.argtypes = [C.POINTER(Segment), C.c_uint32, C.c_uint64, C.POINTER(HParams)]
        L.orc_destroy.argtypes = [C.c_void_p]
        L.orc_set_lr.argtypes = [C.c_void_p, C.c_float]
        L.orc_step.restype = C.c_int
        L.orc_step.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64]
        L.orc_get_layers.argtypes = [C.c_void_p, C.POINTER(Layer)]
        L.orc_get_status.argtypes = [C.c_void_p, C.POINTER(Status)]
        L.orc_get_momentum.argtypes = [C.c_void_p, C.c_void_p]
        L.orc_get_mask.argtypes = [C.c_void_p, C.c_void_p]
        L.orc_mask_words.restype = C.c_uint64
        L.orc_mask_words.argtypes = [C.c_void_p]
        L.orc_sizeof_layer.restype = C.c_uint64
        L.orc_philox4x32_10.argtypes = [C.POINTER(C.c_uint32), C.POINTER(C.c_uint32), C.POINTER(C.c_uint32)]
        L.orc_rademacher_bit.restype = C.c_uint32
        L.orc_rademacher_bit.argtypes = [C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint64]
        L.orc_probe.argtypes = [C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint64, C.c_uint64, C.c_void_p]
        L.orc_moments.argtypes = [C.c_void_p, C.c_uint64, C.POINTER(C.c_double), C.POINTER(C.c_double)]
        L.orc_cast_array.argtypes = [C.c_void_p, C.c_uint64, C.c_uint32, C.c_void_p]
        L.orc_hutchinson_abs.argtypes = [C.c_void_p, C.c_uint64, C.c_uint32, C.c_uint64, C.c_uint64,
                                         C.c_uint64, C.c_uint64, C.c_void_p]
        L.orc_power_iterate.argtypes = [C.POINTER(Segment), C.c_uint32, C.c_uint64, C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_batch_next.restype = C.c_int64
        L.orc_batch_next.argtypes = [C.c_int64, C.c_int64, C.c_int64, C.c_double, C.c_double,
                                     C.c_double, C.c_double, C.c_int64, C.c_int64]
        assert L.orc_sizeof_layer() == C.sizeof(Layer)
        _lib = L
    return _lib


def _ptr(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def philox4x32_10(ctr, key):
    c = (C.c_uint32 * 4)(*ctr)
    k = (C.c_uint32 * 2)(*key)
    o = (C.c_uint32 * 4)()
    lib().orc_philox4x32_10(c, k, o)
    return tuple(int(x) for x in o)


def rademacher_bit(seed, t, p, i):
    return int(lib().orc_rademacher_bit(seed, t, p, i))


def probe(seed, t, p, first, n):
    """z for flat elements [first, first+n) as float32 +-1."""
    z = np.empty(n, dtype=np.float32)
    lib().orc_probe(seed, t, p, first, n, _ptr(z))
    return z


def moments(x):
    x = np.ascontiguousarray(x, dtype=np.float32)
    m, v = C.c_double(), C.c_double()
    lib().orc_moments(_ptr(x), x.size, C.byref(m), C.byref(v))
    return m.value, v.value


def cast(x, to_bf16):
    """float32 array -> uint16 bit patterns of bfloat16 (to_bf16) or binary16."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.size, dtype=np.uint16)
    lib().orc_cast_array(_ptr(x), x.size, 1 if to_bf16 else 0, _ptr(out))
    return out


def hutchinson_abs(hz, n_total, P, seed, t, offset, length):
    hz = np.ascontiguousarray(hz, dtype=np.float32)
    assert hz.size == P * n_total
    a = np.empty(length, dtype=np.float32)
    lib().orc_hutchinson_abs(_ptr(hz), n_total, P, seed, t, offset, length, _ptr(a))
    return a


def power_iterate(table, n_total, u, hu, v=None, lam_v=None):
    """One power-iteration step per layer. v: [m, n_total] or None; lam_v: [m, L] or None.
    Returns (u_next [n_total], lambda [L], norm [L]); elements outside the layers of u_next are 0."""
    L = len(table)
    segs = (Segment * L)(*[Segment(int(o), int(n)) for o, n in table])
    u = np.ascontiguousarray(u, dtype=np.float32)
    hu = np.ascontiguousarray(hu, dtype=np.float32)
    m = 0 if v is None else int(np.asarray(v).shape[0])
    if m:
        v = np.ascontiguousarray(v, dtype=np.float32).reshape(m, n_total)
        lam_v = np.ascontiguousarray(lam_v, dtype=np.float32).reshape(m, L)
    out = np.zeros(n_total, dtype=np.float32)
    lam = np.zeros(L, dtype=np.float32)
    nrm = np.zeros(L, dtype=np.float32)
    lib().orc_power_iterate(segs, L, n_total, _ptr(u), _ptr(hu), _ptr(v) if m else None, _ptr(lam_v) if m else None, m,
                            _ptr(out), _ptr(lam), _ptr(nrm))
    return out, lam, nrm


def batch_next(B, delta_up, delta_down, rho_low, rho_high, mem_usage, mem_max, B_min, B_max):
    return int(lib().orc_batch_next(B, delta_up, delta_down, rho_low, rho_high, mem_usage, mem_max, B_min, B_max))


class Oracle:
    """Per-layer optimizer state plus the step, on the host."""

    def __init__(self, table, n_total, beta=0.9, tau_low=1e-7, tau_high=1e-5, tau_curv=0.9, alpha=1.0,
                 eta0=0.1, topk_ppm=1000000, num_probes=1, t_ctrl=1, grad_dtype="f32", momentum=0.0, weight_decay=0.0):
        self.L = len(table)
        self.n_total = int(n_total)
        segs = (Segment * self.L)(*[Segment(int(o), int(n)) for o, n in table])
        self.hp = HParams(beta, tau_low, tau_high, tau_curv, alpha, eta0, topk_ppm, num_probes, t_ctrl,
                          1 if grad_dtype == "bf16" else 0, momentum, weight_decay)
        self.grad_bf16 = grad_dtype == "bf16"
        self._h = lib().orc_create(segs, self.L, self.n_total, C.byref(self.hp))
        if not self._h:
            raise ValueError("oracle: invalid segment table or hyper-parameters")

    def __del__(self):
        if getattr(self, "_h", None):
            lib().orc_destroy(self._h)
            self._h = None

    def set_lr(self, eta0):
        lib().orc_set_lr(self._h, eta0)

    def step(self, w, g, hz, c, seed, t):
        """w float32 [n_total] (in place); g float32 or uint16(bf16 bits); hz float32 [P*n_total] or None;
        c uint16 [n_total] (in place). Returns True when the step was skipped (non-finite input)."""
        assert w.dtype == np.float32 and w.size == self.n_total and w.flags.c_contiguous
        assert c.dtype == np.uint16 and c.size == self.n_total and c.flags.c_contiguous
        assert g.dtype == (np.uint16 if self.grad_bf16 else np.float32) and g.size == self.n_total
        if hz is not None:
            assert hz.dtype == np.float32 and hz.size == self.hp.num_probes * self.n_total
        return bool(lib().orc_step(self._h, _ptr(w), _ptr(g), _ptr(hz), _ptr(c), seed, t))

    def layers(self):
        arr = (Layer * self.L)()
        lib().orc_get_layers(self._h, arr)
        return list(arr)

    def status(self):
        s = Status()
        lib().orc_get_status(self._h, C.byref(s))
        return s

    def mask(self):
        n = lib().orc_mask_words(self._h)
        m = np.zeros(n, dtype=np.uint32)
        lib().orc_get_mask(self._h, _ptr(m))
        return m

    def momentum_buffer(self):
        m = np.zeros(self.n_total, dtype=np.float32)
        lib().orc_get_momentum(self._h, _ptr(m))
        return m

    def codes(self):
        return np.array([ly.code for ly in self.layers()], dtype=np.uint8)
