"""ctypes binding of the C-ABI library (include/hadfl.h): same names, argument marshalling only.

Every step of the path runs inside libhadfl.so (CUDA kernels for sm_100a plus the host planning
arithmetic).  There is no Python or CPU implementation behind these calls: if the library is not
built or cannot be loaded, `lib()` raises.
"""
import ctypes as C
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
# HADFL_LIBRARY names another build of the same library to load instead (the debug build,
# libhadfl_debug.so: same entry points, bounds-checked kernels).
LIB_PATH = os.environ.get("HADFL_LIBRARY") or os.path.join(HERE, "libhadfl.so")

OK, ERR_INVALID, ERR_CUDA, ERR_STATE, ERR_TOO_LARGE = 0, 1, 2, 3, 4
MAX_DEVICES = 32
DTYPE_FP32, DTYPE_BF16 = 0, 1
WEIGHTS_UNIFORM, WEIGHTS_VERSION = 0, 1
ROUND_NEAREST, ROUND_STOCHASTIC = 0, 1


class hadfl_config(C.Structure):
    _fields_ = [
        ("n_devices", C.c_int32),
        ("n_params", C.c_int64),
        ("dtype", C.c_int32),
        ("momentum", C.c_float),
        ("weight_decay", C.c_float),
        ("grad_std", C.c_float),
        ("init_std", C.c_float),
        ("seed", C.c_uint64),
        ("version_scale", C.c_double),
        ("weight_mode", C.c_int32),
        ("w_ptr", C.c_void_p),
        ("m_ptr", C.c_void_p),
        ("row_stride_elems", C.c_int64),
        ("cuda_stream", C.c_void_p),
        ("m_dtype", C.c_int32),
        ("rounding", C.c_int32),
    ]


class HadflError(RuntimeError):
    def __init__(self, what, code, cuda_error=0):
        names = {ERR_INVALID: "HADFL_ERR_INVALID", ERR_CUDA: "HADFL_ERR_CUDA", ERR_STATE: "HADFL_ERR_STATE",
                 ERR_TOO_LARGE: "HADFL_ERR_TOO_LARGE"}
        msg = "%s failed: %s" % (what, names.get(code, str(code)))
        if code == ERR_CUDA:
            msg += " (cudaError %d)" % cuda_error
        super().__init__(msg)
        self.code = code
        self.cuda_error = cuda_error


_lib = None
_i32p, _u32p, _u64p = C.POINTER(C.c_int32), C.POINTER(C.c_uint32), C.POINTER(C.c_uint64)
_u8p, _f32p, _f64p = C.POINTER(C.c_uint8), C.POINTER(C.c_float), C.POINTER(C.c_double)
_H = C.c_void_p

# Every symbol include/hadfl.h declares: name -> (result type, argument types).
SIGNATURES = {
    "hadfl_init": (C.c_int, [C.POINTER(hadfl_config), C.POINTER(_H)]),
    "hadfl_destroy": (C.c_int, [_H]),
    "hadfl_local_step": (C.c_int, [_H, _i32p, _i32p, C.c_int32, C.c_float]),
    "hadfl_select": (C.c_int, [_H, C.c_int64, _f64p, C.c_uint64, C.c_int32, _i32p]),
    "hadfl_select_probs": (C.c_int, [_H, _f64p, _f64p]),
    "hadfl_select_probs_after": (C.c_int, [_H, _i32p, _i32p, C.c_int32, _f64p]),
    "hadfl_aggregate": (C.c_int, [_H, _i32p, C.c_int32, _f64p]),
    "hadfl_aggregation_weights": (C.c_int, [_H, _i32p, C.c_int32, _f64p, _f32p]),
    "hadfl_broadcast": (C.c_int, [_H, C.c_int32, _i32p, C.c_int32]),
    "hadfl_integrate": (C.c_int, [_H, C.c_int32, _i32p, C.c_int32, C.c_float]),
    "hadfl_set_sync_beta": (C.c_int, [_H, C.c_float]),
    "hadfl_round": (C.c_int, [_H, _i32p, _i32p, C.c_int32, C.c_float, C.c_int64, _f64p, C.c_uint64, C.c_int32,
                              C.c_int32, _i32p]),
    "hadfl_rounds": (C.c_int, [_H, C.c_int64, C.c_int32, _i32p, C.c_float, C.c_uint64, C.c_int32, C.c_int32, _i32p]),
    "hadfl_stats_enqueue": (C.c_int, [_H, C.c_int32]),
    "hadfl_stats_read": (C.c_int, [_H, _f32p, _f32p]),
    "hadfl_stats": (C.c_int, [_H, C.c_int32, _f32p, _f32p]),
    "hadfl_stats_noalloc": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_int64, C.c_int64, C.c_int32,
                                      C.c_void_p, C.c_void_p]),
    "hadfl_stats_grid_lanes": (C.c_int64, [C.c_int32, C.c_int32, C.c_int64, C.c_int32, C.c_int64]),
    "hadfl_read_params": (C.c_int, [_H, C.c_int32, C.c_void_p, C.c_int64]),
    "hadfl_read_momentum": (C.c_int, [_H, C.c_int32, C.c_void_p, C.c_int64]),
    "hadfl_write_params": (C.c_int, [_H, C.c_int32, C.c_void_p, C.c_int64]),
    "hadfl_write_momentum": (C.c_int, [_H, C.c_int32, C.c_void_p, C.c_int64]),
    "hadfl_backup_begin": (C.c_int, [_H, C.c_int32, C.c_void_p, C.c_int64]),
    "hadfl_backup_wait": (C.c_int, [_H]),
    "hadfl_get_versions": (C.c_int, [_H, _u32p, _u64p]),
    "hadfl_set_versions": (C.c_int, [_H, _u32p, _u64p]),
    "hadfl_set_available": (C.c_int, [_H, _u8p]),
    "hadfl_synchronize": (C.c_int, [_H]),
    "hadfl_last_cuda_error": (C.c_int, [_H]),
    "hadfl_launch_count": (C.c_uint64, [_H]),
    "hadfl_row_stride": (C.c_int64, [_H]),
    "hadfl_round_grid": (C.c_int32, [_H]),
    "hadfl_set_round_batch": (C.c_int, [_H, C.c_int32]),
    "hadfl_round_batch": (C.c_int32, [_H]),
    "hadfl_last_round_pack": (C.c_int32, [_H]),
    "hadfl_stats_read_round": (C.c_int, [_H, C.c_int32, _f32p, _f32p]),
    "hadfl_selection_probs": (C.c_int, [_f64p, _u8p, C.c_int32, _f64p]),
    "hadfl_selection_draw": (C.c_int, [_f64p, _u8p, C.c_int32, C.c_int64, C.c_uint64, C.c_int32, _i32p]),
    "hadfl_predict_version": (C.c_int, [_f64p, C.c_int32, C.c_double, C.c_double, _f64p]),
    "hadfl_debug_build": (C.c_int, []),
    "hadfl_debug_check": (C.c_int, [_H, _u64p]),
    "hadfl_debug_range_holds": (C.c_int, [C.c_uint64, C.c_uint64, C.c_uint64, C.c_uint64]),
    "hadfl_debug_philox": (C.c_int, [_H, _u32p, _u32p, C.c_int64, _u32p]),
    "hadfl_debug_normals": (C.c_int, [_H, C.c_int32, _u32p, C.c_int64, C.c_uint64, C.c_uint32, _f32p]),
}
SYMBOLS = sorted(SIGNATURES)


def lib():
    """Loads libhadfl.so (never builds it, never substitutes anything for it)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("libhadfl.so is not built: run `python -m paper_2111_08274_b200.build` "
                              "(needs nvcc); there is no fallback implementation")
        l = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            f = getattr(l, name)
            f.restype, f.argtypes = res, args
        _lib = l
    return _lib


def _p(a, ctype):
    return None if a is None else a.ctypes.data_as(C.POINTER(ctype))


def _arr(x, dtype):
    return None if x is None else np.ascontiguousarray(np.asarray(x, dtype=dtype))


# ---- host-only functions -----------------------------------------------------------------------
def hadfl_selection_probs(x, avail=None):
    x, a = _arr(x, np.float64), _arr(avail, np.uint8)
    out = np.empty(len(x), dtype=np.float64)
    rc = lib().hadfl_selection_probs(_p(x, C.c_double), _p(a, C.c_uint8), len(x), _p(out, C.c_double))
    if rc:
        raise HadflError("hadfl_selection_probs", rc)
    return out


def hadfl_selection_draw(x, k, round_, seed, avail=None):
    x, a = _arr(x, np.float64), _arr(avail, np.uint8)
    out = np.empty(max(int(k), 1), dtype=np.int32)
    rc = lib().hadfl_selection_draw(_p(x, C.c_double), _p(a, C.c_uint8), len(x), round_, seed, k,
                                    _p(out, C.c_int32))
    if rc:
        raise HadflError("hadfl_selection_draw", rc)
    return out[:k]


def hadfl_predict_version(series, alpha, m=1.0):
    s = _arr(series, np.float64)
    out = C.c_double(0.0)
    rc = lib().hadfl_predict_version(_p(s, C.c_double), len(s), alpha, m, C.byref(out))
    if rc:
        raise HadflError("hadfl_predict_version", rc)
    return out.value


def hadfl_stats_noalloc(w_ptr, dtype, n_devices, n_params, row_stride_elems, ref_device,
                        out_stats_ptr, stream=0):
    """Statistics for callers that must not allocate: raw DEVICE addresses in, status code out
    (see include/hadfl.h).  out_stats_ptr: 2N device floats, norm2 then div2.  Asynchronous."""
    return int(lib().hadfl_stats_noalloc(w_ptr, dtype, n_devices, n_params, row_stride_elems,
                                         ref_device, out_stats_ptr, stream or None))


def hadfl_debug_build():
    return bool(lib().hadfl_debug_build())


def hadfl_debug_range_holds(lo, hi, addr, nbytes):
    return bool(lib().hadfl_debug_range_holds(lo, hi, addr, nbytes))


def hadfl_stats_grid_lanes(sm_count, n_devices, n_params, dtype=DTYPE_FP32, max_blocks=0):
    """Blocks per row of a statistics launch on a GPU with sm_count SMs (host only)."""
    return int(lib().hadfl_stats_grid_lanes(sm_count, n_devices, n_params, dtype, max_blocks))


# ---- the handle --------------------------------------------------------------------------------
class Hadfl:
    """One arena of N replicas on the current CUDA device.  Method names are the C entry points
    without the `hadfl_` prefix.

    w_ptr / m_ptr: device addresses of caller-owned arenas (e.g. torch tensors' data_ptr(); the
    tensors must outlive this object), or None to let the library allocate.  stream: a
    cudaStream_t value (e.g. torch.cuda.current_stream().cuda_stream)."""

    def __init__(self, n_devices, n_params, dtype=DTYPE_FP32, momentum=0.9, weight_decay=5e-4,
                 grad_std=1e-3, init_std=0.05, seed=0, version_scale=1.0, weight_mode=0,
                 w_ptr=None, m_ptr=None, row_stride_elems=0, stream=0, m_dtype=DTYPE_FP32,
                 rounding=ROUND_NEAREST):
        self._lib = lib()
        self.n_devices, self.n_params, self.dtype = int(n_devices), int(n_params), int(dtype)
        cfg = hadfl_config(n_devices, n_params, dtype, momentum, weight_decay, grad_std, init_std,
                           seed, version_scale, weight_mode, w_ptr, m_ptr, row_stride_elems,
                           stream or None, m_dtype, rounding)
        h = _H()
        rc = self._lib.hadfl_init(C.byref(cfg), C.byref(h))
        self._h = h if h.value else None
        if rc:
            err = self._lib.hadfl_last_cuda_error(self._h) if self._h else 0
            self.destroy()
            raise HadflError("hadfl_init", rc, err)

    @classmethod
    def from_workload(cls, wl, **kw):
        return cls(wl.n_devices, wl.n_params, dtype=wl.dtype, momentum=wl.momentum,
                   weight_decay=wl.weight_decay, grad_std=wl.grad_std, init_std=wl.init_std,
                   seed=wl.seed, version_scale=wl.version_scale, weight_mode=wl.weight_mode,
                   m_dtype=wl.m_dtype, rounding=wl.rounding, **kw)

    def _check(self, rc, what):
        if rc:
            raise HadflError(what, rc, self._lib.hadfl_last_cuda_error(self._h))

    def destroy(self):
        if getattr(self, "_h", None):
            self._lib.hadfl_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def local_step(self, device_ids, steps, lr):
        ids, st = _arr(device_ids, np.int32), _arr(steps, np.int32)
        if len(ids) != len(st):
            raise HadflError("hadfl_local_step", ERR_INVALID)
        self._check(self._lib.hadfl_local_step(self._h, _p(ids, C.c_int32), _p(st, C.c_int32),
                                               len(ids), lr), "hadfl_local_step")

    def select(self, round_, k, seed, versions=None):
        v = _arr(versions, np.float64)
        out = np.empty(max(int(k), 1), dtype=np.int32)
        self._check(self._lib.hadfl_select(self._h, round_, _p(v, C.c_double), seed, k,
                                           _p(out, C.c_int32)), "hadfl_select")
        return out[:k]

    def select_probs(self, versions=None):
        v = _arr(versions, np.float64)
        out = np.empty(self.n_devices, dtype=np.float64)
        self._check(self._lib.hadfl_select_probs(self._h, _p(v, C.c_double), _p(out, C.c_double)),
                    "hadfl_select_probs")
        return out

    def select_probs_after(self, device_ids, steps):
        ids, st = _arr(device_ids, np.int32), _arr(steps, np.int32)
        if len(ids) != len(st):
            raise HadflError("hadfl_select_probs_after", ERR_INVALID)
        out = np.empty(self.n_devices, dtype=np.float64)
        self._check(self._lib.hadfl_select_probs_after(self._h, _p(ids, C.c_int32), _p(st, C.c_int32),
                                                       len(ids), _p(out, C.c_double)),
                    "hadfl_select_probs_after")
        return out

    def aggregate(self, selected, versions=None):
        sel, v = _arr(selected, np.int32), _arr(versions, np.float64)
        self._check(self._lib.hadfl_aggregate(self._h, _p(sel, C.c_int32), len(sel),
                                              _p(v, C.c_double)), "hadfl_aggregate")

    def aggregation_weights(self, selected, versions=None):
        sel, v = _arr(selected, np.int32), _arr(versions, np.float64)
        out = np.empty(max(len(sel), 1), dtype=np.float32)
        self._check(self._lib.hadfl_aggregation_weights(self._h, _p(sel, C.c_int32), len(sel),
                                                        _p(v, C.c_double), _p(out, C.c_float)),
                    "hadfl_aggregation_weights")
        return out[: len(sel)]

    def broadcast(self, src, dst_ids):
        dst = _arr(dst_ids, np.int32)
        self._check(self._lib.hadfl_broadcast(self._h, src, _p(dst, C.c_int32), len(dst)),
                    "hadfl_broadcast")

    def integrate(self, src, dst_ids, beta):
        dst = _arr(dst_ids, np.int32)
        self._check(self._lib.hadfl_integrate(self._h, src, _p(dst, C.c_int32), len(dst), beta),
                    "hadfl_integrate")

    def set_sync_beta(self, beta):
        self._check(self._lib.hadfl_set_sync_beta(self._h, beta), "hadfl_set_sync_beta")

    def round(self, device_ids, steps, lr, round_, k, seed, versions=None, sync_all=False):
        ids, st, v = _arr(device_ids, np.int32), _arr(steps, np.int32), _arr(versions, np.float64)
        if len(ids) != len(st):
            raise HadflError("hadfl_round", ERR_INVALID)
        out = np.empty(max(int(k), 1), dtype=np.int32)
        self._check(self._lib.hadfl_round(self._h, _p(ids, C.c_int32), _p(st, C.c_int32), len(ids), lr,
                                          round_, _p(v, C.c_double), seed, k, 1 if sync_all else 0,
                                          _p(out, C.c_int32)), "hadfl_round")
        return out[:k]

    def rounds(self, first_round, steps, lr, k, seed, sync_every=0):
        """steps: [n_rounds, N] step counts.  Returns the selected ids, [n_rounds, k]."""
        st = np.ascontiguousarray(np.asarray(steps, dtype=np.int32))
        if st.ndim != 2 or st.shape[1] != self.n_devices:
            raise HadflError("hadfl_rounds", ERR_INVALID)
        out = np.empty((st.shape[0], max(int(k), 1)), dtype=np.int32)
        self._check(self._lib.hadfl_rounds(self._h, first_round, st.shape[0], _p(st, C.c_int32), lr, seed,
                                           k, sync_every, _p(out, C.c_int32)), "hadfl_rounds")
        return out[:, :k]

    def stats_enqueue(self, ref_device):
        self._check(self._lib.hadfl_stats_enqueue(self._h, ref_device), "hadfl_stats_enqueue")

    def stats_read(self):
        n2 = np.empty(self.n_devices, dtype=np.float32)
        d2 = np.empty(self.n_devices, dtype=np.float32)
        self._check(self._lib.hadfl_stats_read(self._h, _p(n2, C.c_float), _p(d2, C.c_float)),
                    "hadfl_stats_read")
        return n2, d2

    def stats_read_round(self, back):
        """Statistics of the round `back` rounds before the last one of the most recent fused launch."""
        n2 = np.empty(self.n_devices, dtype=np.float32)
        d2 = np.empty(self.n_devices, dtype=np.float32)
        self._check(self._lib.hadfl_stats_read_round(self._h, back, _p(n2, C.c_float), _p(d2, C.c_float)),
                    "hadfl_stats_read_round")
        return n2, d2

    def stats(self, ref_device):
        n2 = np.empty(self.n_devices, dtype=np.float32)
        d2 = np.empty(self.n_devices, dtype=np.float32)
        self._check(self._lib.hadfl_stats(self._h, ref_device, _p(n2, C.c_float), _p(d2, C.c_float)),
                    "hadfl_stats")
        return n2, d2

    def _read(self, fn, name, device_id, count, out):
        count = self.n_params if count is None else int(count)
        if out is None:
            out = np.empty(count, dtype=np.float32)
            ptr = out.ctypes.data
        elif isinstance(out, np.ndarray):
            ptr = out.ctypes.data
        else:                                   # a (pinned) host torch tensor
            ptr = out.data_ptr()
        self._check(fn(self._h, device_id, ptr, count), name)
        return out

    def read_params(self, device_id, count=None, out=None):
        return self._read(self._lib.hadfl_read_params, "hadfl_read_params", device_id, count, out)

    def read_momentum(self, device_id, count=None, out=None):
        return self._read(self._lib.hadfl_read_momentum, "hadfl_read_momentum", device_id, count, out)

    def backup_begin(self, device_id, out, count=None):
        """out: a host buffer of at least `count` floats that stays alive until backup_wait (a
        pinned torch tensor or a numpy array)."""
        count = self.n_params if count is None else int(count)
        ptr = out.ctypes.data if isinstance(out, np.ndarray) else out.data_ptr()
        self._check(self._lib.hadfl_backup_begin(self._h, device_id, ptr, count), "hadfl_backup_begin")

    def backup_wait(self):
        self._check(self._lib.hadfl_backup_wait(self._h), "hadfl_backup_wait")

    def write_params(self, device_id, values):
        v = _arr(values, np.float32)
        self._check(self._lib.hadfl_write_params(self._h, device_id, v.ctypes.data, v.size),
                    "hadfl_write_params")

    def write_momentum(self, device_id, values):
        v = _arr(values, np.float32)
        self._check(self._lib.hadfl_write_momentum(self._h, device_id, v.ctypes.data, v.size),
                    "hadfl_write_momentum")

    def get_versions(self):
        v = np.empty(self.n_devices, dtype=np.uint32)
        s = np.empty(self.n_devices, dtype=np.uint64)
        self._check(self._lib.hadfl_get_versions(self._h, _p(v, C.c_uint32), _p(s, C.c_uint64)),
                    "hadfl_get_versions")
        return v, s

    def set_versions(self, versions=None, step_counts=None):
        v, s = _arr(versions, np.uint32), _arr(step_counts, np.uint64)
        self._check(self._lib.hadfl_set_versions(self._h, _p(v, C.c_uint32), _p(s, C.c_uint64)),
                    "hadfl_set_versions")

    def set_available(self, mask=None):
        m = _arr(mask, np.uint8)
        self._check(self._lib.hadfl_set_available(self._h, _p(m, C.c_uint8)), "hadfl_set_available")

    def synchronize(self):
        self._check(self._lib.hadfl_synchronize(self._h), "hadfl_synchronize")

    def debug_check(self):
        """Raises HadflError (HADFL_ERR_STATE) if, in the debug build, a kernel skipped an out-of-range access."""
        bad = C.c_uint64(0)
        rc = self._lib.hadfl_debug_check(self._h, C.byref(bad))
        if rc:
            raise HadflError("hadfl_debug_check (first bad address 0x%x)" % bad.value, rc,
                             self._lib.hadfl_last_cuda_error(self._h))

    def launch_count(self):
        return int(self._lib.hadfl_launch_count(self._h))

    def row_stride(self):
        return int(self._lib.hadfl_row_stride(self._h))

    def round_grid(self):
        return int(self._lib.hadfl_round_grid(self._h))

    def set_round_batch(self, max_rounds):
        self._check(self._lib.hadfl_set_round_batch(self._h, max_rounds), "hadfl_set_round_batch")

    def round_batch(self):
        return int(self._lib.hadfl_round_batch(self._h))

    def last_round_pack(self):
        return int(self._lib.hadfl_last_round_pack(self._h))

    def debug_philox(self, counters, key):
        c = _arr(counters, np.uint32).reshape(-1, 4)
        k = _arr(key, np.uint32)
        out = np.empty_like(c)
        self._check(self._lib.hadfl_debug_philox(self._h, _p(c, C.c_uint32), _p(k, C.c_uint32),
                                                 c.shape[0], _p(out, C.c_uint32)), "hadfl_debug_philox")
        return out

    def debug_normals(self, which, groups, step=0, device=0):
        g = _arr(groups, np.uint32)
        out = np.empty((g.size, 4), dtype=np.float32)
        self._check(self._lib.hadfl_debug_normals(self._h, which, _p(g, C.c_uint32), g.size, step,
                                                  device, _p(out, C.c_float)), "hadfl_debug_normals")
        return out
