"""CPU oracle for the HADFL round hot path: TEST INFRASTRUCTURE ONLY.

A ctypes front for oracle/hadfl_oracle.cpp (single-threaded C++, written from the paper:
Eq. 3 / Algorithm 1 local update, Eq. 5 partial aggregation, Eq. 8 selection, Eq. 7 version
prediction).  Only tests, the smoke check and the benchmark's CPU-baseline leg may import it;
the CUDA library and its Python binding never do, and share no code with it.
"""
import ctypes as C
import numpy as np

from . import build as _build

_lib = None
_lib_omp = None


def lib(openmp=False):
    """The oracle library: the plain single-threaded build, or (openmp=True) the build of the same
    source with -fopenmp that the all-cores CPU baseline times."""
    global _lib, _lib_omp
    if openmp:
        if _lib_omp is None:
            _lib_omp = C.CDLL(_build.build(openmp=True))
            _declare(_lib_omp)
        return _lib_omp
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _declare(_lib)
    return _lib


def threads(openmp=False):
    """Threads the simulation loops of that build run on (1 for the plain build)."""
    return int(lib(openmp).oracle_threads())


_u32p = C.POINTER(C.c_uint32)
_u64p = C.POINTER(C.c_uint64)
_i32p = C.POINTER(C.c_int32)
_u8p = C.POINTER(C.c_uint8)
_f32p = C.POINTER(C.c_float)
_f64p = C.POINTER(C.c_double)


def _declare(l):
    l.oracle_threads.argtypes = []
    l.oracle_threads.restype = C.c_int
    l.oracle_philox4x32_10.argtypes = [_u32p, _u32p, _u32p]
    l.oracle_philox4x32_10.restype = None
    l.oracle_words_to_normals.argtypes = [_u32p, _f64p]
    l.oracle_words_to_normals.restype = None
    l.oracle_grad_normals.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64, C.c_uint32, _f32p]
    l.oracle_grad_normals.restype = None
    l.oracle_init_normals.argtypes = [C.c_uint64, C.c_uint32, _f32p]
    l.oracle_init_normals.restype = None
    l.oracle_select_bits.argtypes = [C.c_uint64, C.c_int64, C.c_uint32]
    l.oracle_select_bits.restype = C.c_uint64
    l.oracle_round_to_bf16.argtypes = [C.c_float]
    l.oracle_round_to_bf16.restype = C.c_float
    l.oracle_round_to_bf16_stochastic.argtypes = [C.c_float, C.c_uint32]
    l.oracle_round_to_bf16_stochastic.restype = C.c_float
    l.oracle_rounding_words.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64, C.c_uint32, _u32p]
    l.oracle_rounding_words.restype = None
    l.oracle_third_quartile.argtypes = [_f64p, C.c_int]
    l.oracle_third_quartile.restype = C.c_double
    l.oracle_select_probs.argtypes = [_f64p, _u8p, C.c_int, _f64p]
    l.oracle_select_probs.restype = None
    l.oracle_select.argtypes = [_f64p, _u8p, C.c_int, C.c_int64, C.c_uint64, C.c_int, _i32p]
    l.oracle_select.restype = C.c_int
    l.oracle_predict_version.argtypes = [_f64p, C.c_int, C.c_double, C.c_double]
    l.oracle_predict_version.restype = C.c_double
    l.oracle_sim_create.argtypes = [C.c_int, C.c_int64, C.c_int, C.c_float, C.c_float, C.c_float,
                                    C.c_float, C.c_uint64, C.c_double, C.c_int, _u32p, C.c_int64,
                                    C.c_int, C.c_int]
    l.oracle_sim_create.restype = C.c_void_p
    l.oracle_sim_destroy.argtypes = [C.c_void_p]
    l.oracle_sim_destroy.restype = None
    l.oracle_sim_n_cols.argtypes = [C.c_void_p]
    l.oracle_sim_n_cols.restype = C.c_int64
    l.oracle_sim_local_step.argtypes = [C.c_void_p, _i32p, _i32p, C.c_int, C.c_float]
    l.oracle_sim_local_step.restype = C.c_int
    l.oracle_sim_select_probs.argtypes = [C.c_void_p, _f64p, _f64p]
    l.oracle_sim_select_probs.restype = C.c_int
    l.oracle_sim_select.argtypes = [C.c_void_p, C.c_int64, _f64p, C.c_uint64, C.c_int, _i32p]
    l.oracle_sim_select.restype = C.c_int
    l.oracle_sim_aggregation_weights.argtypes = [C.c_void_p, _i32p, C.c_int, _f64p, _f32p]
    l.oracle_sim_aggregation_weights.restype = C.c_int
    l.oracle_sim_aggregate.argtypes = [C.c_void_p, _i32p, C.c_int, _f64p]
    l.oracle_sim_aggregate.restype = C.c_int
    l.oracle_sim_broadcast.argtypes = [C.c_void_p, C.c_int, _i32p, C.c_int]
    l.oracle_sim_broadcast.restype = C.c_int
    l.oracle_sim_integrate.argtypes = [C.c_void_p, C.c_int, _i32p, C.c_int, C.c_float]
    l.oracle_sim_integrate.restype = C.c_int
    l.oracle_sim_stats.argtypes = [C.c_void_p, C.c_int, _f64p, _f64p]
    l.oracle_sim_stats.restype = C.c_int
    l.oracle_sim_read.argtypes = [C.c_void_p, C.c_int, C.c_int, _f32p]
    l.oracle_sim_read.restype = C.c_int
    l.oracle_sim_write.argtypes = [C.c_void_p, C.c_int, C.c_int, _f32p]
    l.oracle_sim_write.restype = C.c_int
    l.oracle_sim_get_versions.argtypes = [C.c_void_p, _u32p, _u64p]
    l.oracle_sim_get_versions.restype = None
    l.oracle_sim_set_versions.argtypes = [C.c_void_p, _u32p, _u64p]
    l.oracle_sim_set_versions.restype = None
    l.oracle_sim_set_available.argtypes = [C.c_void_p, _u8p]
    l.oracle_sim_set_available.restype = None


def _ptr(a, ctype):
    return a.ctypes.data_as(C.POINTER(ctype)) if a is not None else None


def _i32(x):
    return np.ascontiguousarray(np.asarray(x, dtype=np.int32))


def _f64(x):
    return None if x is None else np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def _u8(x):
    return None if x is None else np.ascontiguousarray(np.asarray(x, dtype=np.uint8))


# ---- generator primitives -----------------------------------------------------------------
def philox4x32_10(ctr, key):
    ctr = np.ascontiguousarray(np.asarray(ctr, dtype=np.uint32))
    key = np.ascontiguousarray(np.asarray(key, dtype=np.uint32))
    out = np.empty(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_ptr(ctr, C.c_uint32), _ptr(key, C.c_uint32), _ptr(out, C.c_uint32))
    return out


def philox4x32_10_many(ctrs, key):
    """ctrs: [n,4] uint32 -> [n,4] uint32 words."""
    ctrs = np.ascontiguousarray(np.asarray(ctrs, dtype=np.uint32))
    key = np.ascontiguousarray(np.asarray(key, dtype=np.uint32))
    out = np.empty_like(ctrs)
    f = lib().oracle_philox4x32_10
    kp = _ptr(key, C.c_uint32)
    base_in, base_out = ctrs.ctypes.data, out.ctypes.data
    for i in range(ctrs.shape[0]):
        f(C.cast(base_in + 16 * i, _u32p), kp, C.cast(base_out + 16 * i, _u32p))
    return out


def words_to_normals(words):
    words = np.ascontiguousarray(np.asarray(words, dtype=np.uint32))
    z = np.empty(4, dtype=np.float64)
    lib().oracle_words_to_normals(_ptr(words, C.c_uint32), _ptr(z, C.c_double))
    return z


def grad_normals(seed, group, step, device):
    z = np.empty(4, dtype=np.float32)
    lib().oracle_grad_normals(seed, group, step, device, _ptr(z, C.c_float))
    return z


def init_normals(seed, group):
    z = np.empty(4, dtype=np.float32)
    lib().oracle_init_normals(seed, group, _ptr(z, C.c_float))
    return z


def select_bits(seed, round_, t):
    return int(lib().oracle_select_bits(seed, round_, t))


def round_to_bf16(v):
    return float(lib().oracle_round_to_bf16(float(v)))


def round_to_bf16_stochastic(v, r16):
    return float(lib().oracle_round_to_bf16_stochastic(float(v), int(r16)))


def rounding_words(seed, group, last_step, device):
    out = np.empty(4, dtype=np.uint32)
    lib().oracle_rounding_words(seed, group, last_step, device, _ptr(out, C.c_uint32))
    return out


# ---- selection / prediction ------------------------------------------------------------------
def third_quartile(x):
    x = _f64(x)
    return float(lib().oracle_third_quartile(_ptr(x, C.c_double), len(x)))


def select_probs(x, avail=None):
    x = _f64(x)
    a = _u8(avail)
    P = np.empty(len(x), dtype=np.float64)
    lib().oracle_select_probs(_ptr(x, C.c_double), _ptr(a, C.c_uint8), len(x), _ptr(P, C.c_double))
    return P


def select(x, k, round_, seed, avail=None):
    x = _f64(x)
    a = _u8(avail)
    out = np.empty(max(k, 1), dtype=np.int32)
    rc = lib().oracle_select(_ptr(x, C.c_double), _ptr(a, C.c_uint8), len(x), round_, seed, k,
                             _ptr(out, C.c_int32))
    if rc != 0:
        raise ValueError("oracle_select rejected its arguments (rc=%d)" % rc)
    return out[:k]


def predict_version(series, alpha, m=1.0):
    v = _f64(series)
    return float(lib().oracle_predict_version(_ptr(v, C.c_double), len(v), alpha, m))


# ---- the simulated system ---------------------------------------------------------------------
class OracleError(ValueError):
    pass


class Sim:
    """N device replicas over all (groups=None) or a subset of the 4-column groups."""

    def __init__(self, n_devices, n_params, dtype=0, momentum=0.9, weight_decay=5e-4,
                 grad_std=1e-2, init_std=0.05, seed=0, version_scale=1.0, weight_mode=0,
                 groups=None, m_dtype=0, rounding=0, openmp=False):
        self.n_devices, self.n_params, self.dtype = n_devices, n_params, dtype
        self.m_dtype, self.rounding = m_dtype, rounding
        if groups is not None:
            groups = np.ascontiguousarray(np.asarray(groups, dtype=np.uint32))
        self.groups = groups
        self._lib = lib(openmp)
        self._h = self._lib.oracle_sim_create(n_devices, n_params, dtype, momentum, weight_decay,
                                          grad_std, init_std, seed, version_scale, weight_mode,
                                          _ptr(groups, C.c_uint32),
                                          0 if groups is None else len(groups), m_dtype, rounding)
        if not self._h:
            raise OracleError("oracle_sim_create rejected its arguments")
        self.n_cols = int(self._lib.oracle_sim_n_cols(self._h))

    def close(self):
        if self._h:
            self._lib.oracle_sim_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc, what):
        if rc != 0:
            raise OracleError("%s rejected its arguments (rc=%d)" % (what, rc))

    def local_step(self, ids, steps, lr):
        ids, steps = _i32(ids), _i32(steps)
        self._check(self._lib.oracle_sim_local_step(self._h, _ptr(ids, C.c_int32), _ptr(steps, C.c_int32),
                                                len(ids), lr), "local_step")

    def select_probs(self, versions=None):
        v = _f64(versions)
        P = np.empty(self.n_devices, dtype=np.float64)
        self._check(self._lib.oracle_sim_select_probs(self._h, _ptr(v, C.c_double), _ptr(P, C.c_double)),
                    "select_probs")
        return P

    def select(self, round_, k, seed, versions=None):
        v = _f64(versions)
        out = np.empty(max(k, 1), dtype=np.int32)
        self._check(self._lib.oracle_sim_select(self._h, round_, _ptr(v, C.c_double), seed, k,
                                            _ptr(out, C.c_int32)), "select")
        return out[:k]

    def aggregation_weights(self, selected, versions=None):
        sel, v = _i32(selected), _f64(versions)
        a = np.empty(len(sel), dtype=np.float32)
        self._check(self._lib.oracle_sim_aggregation_weights(self._h, _ptr(sel, C.c_int32), len(sel),
                                                         _ptr(v, C.c_double), _ptr(a, C.c_float)),
                    "aggregation_weights")
        return a

    def aggregate(self, selected, versions=None):
        sel, v = _i32(selected), _f64(versions)
        self._check(self._lib.oracle_sim_aggregate(self._h, _ptr(sel, C.c_int32), len(sel),
                                               _ptr(v, C.c_double)), "aggregate")

    def broadcast(self, src, dst):
        dst = _i32(dst)
        self._check(self._lib.oracle_sim_broadcast(self._h, src, _ptr(dst, C.c_int32), len(dst)),
                    "broadcast")

    def integrate(self, src, dst, beta):
        dst = _i32(dst)
        self._check(self._lib.oracle_sim_integrate(self._h, src, _ptr(dst, C.c_int32), len(dst), beta),
                    "integrate")

    def stats(self, ref):
        n2 = np.empty(self.n_devices, dtype=np.float64)
        d2 = np.empty(self.n_devices, dtype=np.float64)
        self._check(self._lib.oracle_sim_stats(self._h, ref, _ptr(n2, C.c_double), _ptr(d2, C.c_double)),
                    "stats")
        return n2, d2

    def _read(self, i, which):
        out = np.empty(self.n_cols, dtype=np.float32)
        self._check(self._lib.oracle_sim_read(self._h, i, which, _ptr(out, C.c_float)), "read")
        return out

    def read_cols(self, i):
        """All held columns (4 per group; lanes beyond n_params read 0)."""
        return self._read(i, 0)

    def read_momentum_cols(self, i):
        return self._read(i, 1)

    def read_params(self, i):
        """Full-model simulations only: the n_params parameters of device i."""
        assert self.groups is None
        return self._read(i, 0)[: self.n_params]

    def read_momentum(self, i):
        assert self.groups is None
        return self._read(i, 1)[: self.n_params]

    def write_params(self, i, values, which=0):
        assert self.groups is None
        buf = np.zeros(self.n_cols, dtype=np.float32)
        buf[: self.n_params] = np.asarray(values, dtype=np.float32)
        self._check(self._lib.oracle_sim_write(self._h, i, which, _ptr(buf, C.c_float)), "write")

    def write_momentum(self, i, values):
        self.write_params(i, values, which=1)

    def write_cols(self, i, values, which=0):
        buf = np.ascontiguousarray(np.asarray(values, dtype=np.float32))
        assert buf.size == self.n_cols
        self._check(self._lib.oracle_sim_write(self._h, i, which, _ptr(buf, C.c_float)), "write")

    def get_versions(self):
        v = np.empty(self.n_devices, dtype=np.uint32)
        s = np.empty(self.n_devices, dtype=np.uint64)
        self._lib.oracle_sim_get_versions(self._h, _ptr(v, C.c_uint32), _ptr(s, C.c_uint64))
        return v, s

    def set_versions(self, versions=None, step_counts=None):
        v = None if versions is None else np.ascontiguousarray(np.asarray(versions, dtype=np.uint32))
        s = None if step_counts is None else np.ascontiguousarray(np.asarray(step_counts, dtype=np.uint64))
        self._lib.oracle_sim_set_versions(self._h, _ptr(v, C.c_uint32), _ptr(s, C.c_uint64))

    def set_available(self, mask=None):
        m = _u8(mask)
        self._lib.oracle_sim_set_available(self._h, _ptr(m, C.c_uint8))
