"""Thin ctypes binding of libtriaccel.so: argument marshalling only.

Every function has the name and the meaning of its C entry point in include/triaccel.h.
Device buffers are torch CUDA tensors (torch is used for device memory and streams only);
host outputs are numpy arrays.  There is no fallback: if the shared library is missing or a
call fails, an exception is raised.
"""
import ctypes as C
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libtriaccel.so")

TA_OK, TA_ERR_ARG, TA_ERR_ALIGN, TA_ERR_STATE, TA_ERR_CUDA, TA_ERR_NOMEM = 0, -1, -2, -3, -4, -5
TA_CODE_FP16, TA_CODE_BF16, TA_CODE_FP32 = 0, 1, 2
TA_GRAD_F32, TA_GRAD_BF16 = 0, 1
TA_FLAG_INPUTS_FINITE, TA_FLAG_NO_ONE_LAUNCH, TA_FLAG_GUARD_WORKSPACES, TA_FLAG_COOPERATIVE_LAUNCH = 1, 2, 4, 8

EXPORTS = ["ta_create", "ta_destroy", "ta_step", "ta_step_host", "ta_set_lr", "ta_probe", "ta_stats",
           "ta_precision_codes", "ta_masks", "ta_launch_count", "ta_last_error", "ta_state_size",
           "ta_state_save", "ta_state_load", "ta_batch_next", "ta_timing_begin", "ta_timing_end",
           "ta_grad_moments_static", "ta_static_last_error", "ta_test_expire_next_wait",
           "ta_power_iterate", "ta_set_curvature", "ta_plan_one_launch", "ta_plan_pipeline", "ta_plan_items",
           "ta_create_shard", "ta_shard_sweep", "ta_shard_apply", "ta_test_check_guards", "ta_path"]


class ta_segment(C.Structure):
    _fields_ = [("offset", C.c_uint64), ("length", C.c_uint64)]


class ta_run(C.Structure):
    _fields_ = [("begin", C.c_uint64), ("length", C.c_uint32), ("layer", C.c_uint32), ("warp", C.c_uint32),
                ("reserved", C.c_uint32)]


class ta_task(C.Structure):
    _fields_ = [("begin", C.c_uint64), ("length", C.c_uint32), ("layer", C.c_uint32), ("kind", C.c_uint32),
                ("reserved", C.c_uint32)]


class ta_hparams(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("beta", C.c_float), ("tau_low", C.c_float), ("tau_high", C.c_float),
                ("tau_curv", C.c_float), ("alpha", C.c_float), ("eta0", C.c_float), ("topk_ppm", C.c_uint32),
                ("num_probes", C.c_uint32), ("t_ctrl", C.c_uint32), ("grad_dtype", C.c_uint32),
                ("momentum", C.c_float), ("weight_decay", C.c_float), ("flags", C.c_uint32)]


class ta_layer_stats(C.Structure):
    _fields_ = [("grad_mean", C.c_float), ("grad_var", C.c_float), ("ema_mean", C.c_float), ("ema_var", C.c_float),
                ("lambda_max", C.c_float), ("topk_threshold", C.c_float), ("topk_mass", C.c_float),
                ("eta_scale", C.c_float), ("k", C.c_uint64), ("code", C.c_uint32), ("near_threshold", C.c_uint32)]


class ta_step_status(C.Structure):
    _fields_ = [("step", C.c_uint64), ("nonfinite_count", C.c_uint64), ("skipped", C.c_uint32),
                ("near_threshold_count", C.c_uint32)]


ta_mem_reader = C.CFUNCTYPE(C.c_int, C.c_void_p, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64))


class ta_batch_ctrl(C.Structure):
    _fields_ = [("B", C.c_int64), ("delta_up", C.c_int64), ("delta_down", C.c_int64), ("B_min", C.c_int64),
                ("B_max", C.c_int64), ("rho_low", C.c_double), ("rho_high", C.c_double),
                ("mem_budget_bytes", C.c_uint64), ("mem_reader", ta_mem_reader), ("user", C.c_void_p)]


class TriAccelError(RuntimeError):
    def __init__(self, code, message):
        super().__init__(f"triaccel error {code}: {message}")
        self.code = code


_lib = None


def lib():
    """Loads libtriaccel.so (built in-tree by paper_2508_16905_b200/build.py). Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2508_16905_b200.build` "
                          "(there is no CPU or PyTorch fallback)")
    L = C.CDLL(LIB_PATH)
    vp, u64, u32 = C.c_void_p, C.c_uint64, C.c_uint32
    L.ta_create.argtypes = [C.POINTER(ta_segment), u32, u64, C.POINTER(ta_hparams), C.POINTER(vp)]
    L.ta_destroy.argtypes = [vp]
    L.ta_step.argtypes = [vp, vp, vp, vp, vp, u64, u64, vp]
    L.ta_step_host.argtypes = [vp, vp, vp, vp, vp, u64, u64, vp]
    L.ta_set_lr.argtypes = [vp, C.c_float]
    L.ta_probe.argtypes = [vp, u64, u64, u32, vp, vp]
    L.ta_stats.argtypes = [vp, C.POINTER(ta_layer_stats), C.POINTER(ta_step_status)]
    L.ta_precision_codes.argtypes = [vp, vp]
    L.ta_masks.argtypes = [vp, C.POINTER(vp), C.POINTER(u64)]
    L.ta_launch_count.argtypes = [vp, C.POINTER(u64)]
    L.ta_last_error.argtypes = [vp]
    L.ta_last_error.restype = C.c_char_p
    L.ta_state_size.argtypes = [vp, C.POINTER(u64)]
    L.ta_state_save.argtypes = [vp, vp, u64]
    L.ta_state_load.argtypes = [vp, vp, u64]
    L.ta_batch_next.argtypes = [C.POINTER(ta_batch_ctrl), C.POINTER(C.c_int64)]
    L.ta_timing_begin.argtypes = [vp, u32]
    L.ta_timing_end.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(u32)]
    L.ta_grad_moments_static.argtypes = [C.POINTER(ta_segment), u32, vp, u32, vp, vp, vp]
    L.ta_test_expire_next_wait.argtypes = [vp]
    L.ta_test_check_guards.argtypes = [vp]
    L.ta_path.argtypes = [vp]
    L.ta_path.restype = C.c_char_p
    L.ta_power_iterate.argtypes = [vp, vp, vp, vp, vp, u32, vp, vp, vp, vp]
    L.ta_set_curvature.argtypes = [vp, vp]
    L.ta_plan_one_launch.argtypes = [C.POINTER(ta_segment), u32, u32, C.POINTER(ta_run), u32, C.POINTER(u32), C.POINTER(u32),
                                     C.POINTER(u32)]
    L.ta_plan_pipeline.argtypes = [C.POINTER(ta_segment), u32, u32, C.POINTER(ta_task), u64, C.POINTER(u64)]
    L.ta_plan_items.argtypes = [C.POINTER(ta_segment), u32, u32, u32, C.POINTER(ta_run), u64, C.POINTER(u64), C.POINTER(u32)]
    L.ta_create_shard.argtypes = [C.POINTER(ta_segment), u32, u64, C.POINTER(ta_hparams), u64, u64, C.POINTER(vp)]
    L.ta_shard_sweep.argtypes = [vp, vp, vp, u64, u64, vp, vp]
    L.ta_shard_apply.argtypes = [vp, vp, vp, vp, vp, u32, vp]
    L.ta_static_last_error.argtypes = []
    L.ta_static_last_error.restype = C.c_char_p
    for name in EXPORTS:
        if name not in ("ta_last_error", "ta_static_last_error", "ta_path"):
            getattr(L, name).restype = C.c_int
    _lib = L
    return L


def _check(rc, h=None):
    if rc != TA_OK:
        raise TriAccelError(rc, (lib().ta_last_error(h) or b"").decode())


def _dev_ptr(t):
    if t is None or isinstance(t, C.c_void_p):      # already marshalled (callers in a hurry wrap their tensors once: dev_ptr)
        return t
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("device buffers must be contiguous CUDA tensors")
    return C.c_void_p(t.data_ptr())


def dev_ptr(t):
    """The device address of a contiguous CUDA tensor, marshalled once, for callers that pass the same buffers to many
    calls (every ta_* function takes it in place of the tensor; the tensor must stay alive)."""
    return _dev_ptr(t)


def _host_ptr(a):
    if a is None:
        return None
    if hasattr(a, "data_ptr"):          # (pinned) host torch tensor
        if a.is_cuda or not a.is_contiguous():
            raise ValueError("host buffers must be contiguous host tensors")
        return C.c_void_p(a.data_ptr())
    return a.ctypes.data_as(C.c_void_p)


def _stream(stream):
    if stream is None:
        import torch
        return C.c_void_p(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, C.c_void_p):
        return stream
    return C.c_void_p(int(stream))


def make_hparams(beta=0.9, tau_low=1e-7, tau_high=1e-5, tau_curv=0.9, alpha=1.0, eta0=0.1, topk_ppm=1000000,
                 num_probes=1, t_ctrl=1, grad_dtype="f32", momentum=0.0, weight_decay=0.0, flags=0):
    gd = {"f32": TA_GRAD_F32, "bf16": TA_GRAD_BF16}[grad_dtype] if isinstance(grad_dtype, str) else int(grad_dtype)
    return ta_hparams(C.sizeof(ta_hparams), beta, tau_low, tau_high, tau_curv, alpha, eta0, topk_ppm, num_probes,
                      t_ctrl, gd, momentum, weight_decay, flags)


class Handle:
    """Owns one ta_handle*; destroyed with the object or by ta_destroy()."""

    def __init__(self, ptr, L, n_total, hp):
        self.ptr, self.L, self.n_total, self.hp = ptr, L, n_total, hp

    def __del__(self):
        if getattr(self, "ptr", None):
            try:
                lib().ta_destroy(self.ptr)
            except TypeError:          # interpreter shutdown: the module's globals are already gone
                pass
            self.ptr = None


def ta_create(table, n_total, hp=None, **hp_kwargs):
    """table: sequence of (offset, length) in elements; hp: ta_hparams or keyword fields."""
    hp = hp if hp is not None else make_hparams(**hp_kwargs)
    L = len(table)
    segs = (ta_segment * max(L, 1))(*[ta_segment(int(o), int(n)) for o, n in table])
    out = C.c_void_p()
    rc = lib().ta_create(segs, L, int(n_total), C.byref(hp), C.byref(out))
    if rc != TA_OK:
        raise TriAccelError(rc, (lib().ta_last_error(None) or b"").decode())
    return Handle(out, L, int(n_total), hp)


RECORD_BYTES = 40          # sizeof(ta_layer_record)


def ta_create_shard(table, n_total, range_lo, range_hi, hp=None, **hp_kwargs):
    """A handle for the flat range [range_lo, range_hi) of a model spread over ranks; table and n_total are the whole model's."""
    hp = hp if hp is not None else make_hparams(**hp_kwargs)
    L = len(table)
    segs = (ta_segment * max(L, 1))(*[ta_segment(int(o), int(n)) for o, n in table])
    out = C.c_void_p()
    rc = lib().ta_create_shard(segs, L, int(n_total), C.byref(hp), int(range_lo), int(range_hi), C.byref(out))
    if rc != TA_OK:
        raise TriAccelError(rc, (lib().ta_last_error(None) or b"").decode())
    return Handle(out, L, int(n_total), hp)


def ta_shard_sweep(h, g_local, Hz_local, probe_seed, step, records_out, stream=None):
    """records_out: CUDA uint8 tensor of L * RECORD_BYTES bytes (8-byte aligned)."""
    _check(lib().ta_shard_sweep(h.ptr, _dev_ptr(g_local), _dev_ptr(Hz_local), int(probe_seed), int(step),
                                _dev_ptr(records_out), _stream(stream)), h.ptr)


def ta_shard_apply(h, w_local, g_local, c_local, records_all, world, stream=None):
    """records_all: CUDA uint8 tensor of world * L * RECORD_BYTES bytes, the ranks' records in rank order."""
    _check(lib().ta_shard_apply(h.ptr, _dev_ptr(w_local), _dev_ptr(g_local), _dev_ptr(c_local), _dev_ptr(records_all),
                                int(world), _stream(stream)), h.ptr)


def ta_destroy(h):
    if h.ptr:
        lib().ta_destroy(h.ptr)
        h.ptr = None


def ta_step(h, w, g, Hz, c, probe_seed, step, stream=None):
    _check(lib().ta_step(h.ptr, _dev_ptr(w), _dev_ptr(g), _dev_ptr(Hz), _dev_ptr(c), int(probe_seed), int(step),
                         _stream(stream)), h.ptr)


def ta_step_host(h, w_host, g_host, Hz_host, c_host, probe_seed, step, stream=None):
    _check(lib().ta_step_host(h.ptr, _host_ptr(w_host), _host_ptr(g_host), _host_ptr(Hz_host), _host_ptr(c_host),
                              int(probe_seed), int(step), _stream(stream)), h.ptr)


def ta_set_lr(h, eta0):
    _check(lib().ta_set_lr(h.ptr, float(eta0)), h.ptr)


def ta_probe(h, probe_seed, step, p, z_out, stream=None):
    _check(lib().ta_probe(h.ptr, int(probe_seed), int(step), int(p), _dev_ptr(z_out), _stream(stream)), h.ptr)


def ta_stats(h):
    """Returns (list of ta_layer_stats, ta_step_status); waits for the last step."""
    arr = (ta_layer_stats * h.L)()
    st = ta_step_status()
    _check(lib().ta_stats(h.ptr, arr, C.byref(st)), h.ptr)
    return list(arr), st


def ta_precision_codes(h):
    out = np.zeros(h.L, dtype=np.uint8)
    _check(lib().ta_precision_codes(h.ptr, out.ctypes.data_as(C.c_void_p)), h.ptr)
    return out


def ta_masks(h):
    """Returns (device address or None, number of 32-bit words)."""
    p, n = C.c_void_p(), C.c_uint64()
    _check(lib().ta_masks(h.ptr, C.byref(p), C.byref(n)), h.ptr)
    return p.value, n.value


def ta_masks_to_host(h):
    """The mask words as a numpy uint32 array (waits for the last step); empty when dense."""
    import torch
    ptr, n = ta_masks(h)
    if not ptr or n == 0:
        return np.zeros(0, dtype=np.uint32)
    torch.cuda.synchronize()
    return _wrap_device_int32(ptr, n).cpu().numpy().view(np.uint32).copy()


def _wrap_device_int32(ptr, n):
    import torch

    class _Arr:
        __cuda_array_interface__ = {"shape": (int(n),), "typestr": "<i4", "data": (int(ptr), False), "version": 3}
    return torch.as_tensor(_Arr(), device="cuda")


def ta_launch_count(h):
    n = C.c_uint64()
    _check(lib().ta_launch_count(h.ptr, C.byref(n)), h.ptr)
    return n.value


def ta_timing_begin(h, max_steps):
    _check(lib().ta_timing_begin(h.ptr, int(max_steps)), h.ptr)


def ta_timing_end(h):
    """Returns (ms_sweep, ms_decide, ms_update, steps) summed over the timed steps."""
    a, b, c, n = C.c_double(), C.c_double(), C.c_double(), C.c_uint32()
    _check(lib().ta_timing_end(h.ptr, C.byref(a), C.byref(b), C.byref(c), C.byref(n)), h.ptr)
    return a.value, b.value, c.value, n.value


def ta_grad_moments_static(table, g, grad_dtype, mean_var, nonfinite=None, stream=None):
    """Per-layer gradient mean / variance through the entry point that allocates nothing.
    table: sequence of (offset, length); g: CUDA tensor (float32 or bfloat16 per grad_dtype);
    mean_var: CUDA float64 tensor [2 * L] (output); nonfinite: CUDA int32 tensor [L] or None."""
    L = len(table)
    segs = (ta_segment * max(L, 1))(*[ta_segment(int(o), int(n)) for o, n in table])
    gd = {"f32": TA_GRAD_F32, "bf16": TA_GRAD_BF16}[grad_dtype] if isinstance(grad_dtype, str) else int(grad_dtype)
    rc = lib().ta_grad_moments_static(segs, L, _dev_ptr(g), gd, _dev_ptr(mean_var), _dev_ptr(nonfinite), _stream(stream))
    if rc != TA_OK:
        raise TriAccelError(rc, (lib().ta_static_last_error() or b"").decode())


def ta_power_iterate(h, u, Hu, V, lambda_V, m, u_next, lambda_out, norm_out=None, stream=None):
    _check(lib().ta_power_iterate(h.ptr, _dev_ptr(u), _dev_ptr(Hu), _dev_ptr(V), _dev_ptr(lambda_V), int(m),
                                  _dev_ptr(u_next), _dev_ptr(lambda_out), _dev_ptr(norm_out), _stream(stream)), h.ptr)


def ta_set_curvature(h, lambda_max):
    a = np.ascontiguousarray(lambda_max, dtype=np.float32)
    if a.size != h.L:
        raise ValueError("one value per layer")
    _check(lib().ta_set_curvature(h.ptr, a.ctypes.data_as(C.c_void_p)), h.ptr)


def ta_plan_one_launch(table, warps):
    """table: sequence of (offset, length). Returns (runs as a list of (begin, length, layer, warp), warps_used, max_rows)."""
    L = len(table)
    segs = (ta_segment * max(L, 1))(*[ta_segment(int(o), int(n)) for o, n in table])
    n, used, rows = C.c_uint32(), C.c_uint32(), C.c_uint32()
    cap = L + int(warps) + 8
    out = (ta_run * cap)()
    rc = lib().ta_plan_one_launch(segs, L, int(warps), out, cap, C.byref(n), C.byref(used), C.byref(rows))
    if rc != TA_OK:
        raise TriAccelError(rc, (lib().ta_last_error(None) or b"").decode())
    return [(r.begin, r.length, r.layer, r.warp) for r in out[:n.value]], used.value, rows.value


def ta_plan_items(table, sm_count, topk=False):
    """The work items of the multi-kernel pass: (items as a list of (begin, length, layer, warp, batch_in_one_layer), item_elems)."""
    L = len(table)
    segs = (ta_segment * max(L, 1))(*[ta_segment(int(o), int(n)) for o, n in table])
    n, elems = C.c_uint64(), C.c_uint32()
    rc = lib().ta_plan_items(segs, L, int(sm_count), 1 if topk else 0, None, 0, C.byref(n), C.byref(elems))
    if rc != TA_OK and n.value == 0:
        raise TriAccelError(rc, (lib().ta_last_error(None) or b"").decode())
    out = (ta_run * max(1, n.value))()
    rc = lib().ta_plan_items(segs, L, int(sm_count), 1 if topk else 0, out, n.value, C.byref(n), C.byref(elems))
    if rc != TA_OK:
        raise TriAccelError(rc, (lib().ta_last_error(None) or b"").decode())
    return [(r.begin, r.length, r.layer, r.warp, r.reserved) for r in out[:n.value]], elems.value


def ta_plan_pipeline(table, with_decisions=True):
    """The task queue of the pipelined pass as a list of (kind, layer, begin, length); kind 0 sweep, 1 apply, 2 both."""
    L = len(table)
    segs = (ta_segment * max(L, 1))(*[ta_segment(int(o), int(n)) for o, n in table])
    n = C.c_uint64()
    rc = lib().ta_plan_pipeline(segs, L, 1 if with_decisions else 0, None, 0, C.byref(n))
    if rc != TA_OK and n.value == 0:
        raise TriAccelError(rc, (lib().ta_last_error(None) or b"").decode())
    out = (ta_task * max(1, n.value))()
    rc = lib().ta_plan_pipeline(segs, L, 1 if with_decisions else 0, out, n.value, C.byref(n))
    if rc != TA_OK:
        raise TriAccelError(rc, (lib().ta_last_error(None) or b"").decode())
    return [(t.kind, t.layer, t.begin, t.length) for t in out[:n.value]]


def ta_path(h):
    return (lib().ta_path(h.ptr) or b"").decode()


def ta_test_check_guards(h):
    _check(lib().ta_test_check_guards(h.ptr), h.ptr)


def ta_test_expire_next_wait(h):
    _check(lib().ta_test_expire_next_wait(h.ptr), h.ptr)


def ta_state_save(h):
    n = C.c_uint64()
    _check(lib().ta_state_size(h.ptr, C.byref(n)), h.ptr)
    buf = np.zeros(n.value, dtype=np.uint8)
    _check(lib().ta_state_save(h.ptr, buf.ctypes.data_as(C.c_void_p), n.value), h.ptr)
    return buf


def ta_state_load(h, buf):
    buf = np.ascontiguousarray(buf, dtype=np.uint8)
    _check(lib().ta_state_load(h.ptr, buf.ctypes.data_as(C.c_void_p), buf.size), h.ptr)


def ta_batch_next(bc):
    """bc: ta_batch_ctrl (updated in place). Returns the next batch size."""
    out = C.c_int64()
    rc = lib().ta_batch_next(C.byref(bc), C.byref(out))
    if rc != TA_OK:
        raise TriAccelError(rc, "ta_batch_next failed")
    return out.value
