"""ctypes binding of the C ABI declared in include/ngc.h (same names, argument marshalling only)."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

NGC_MAX_N = 128
NGC_LSQ, NGC_LOGISTIC, NGC_SOFTMAX, NGC_MLP = 0, 1, 2, 3
NGC_F32, NGC_BF16, NGC_F64 = 0, 1, 2
_KINDS = {"lsq": NGC_LSQ, "logistic": NGC_LOGISTIC, "softmax": NGC_SOFTMAX, "mlp": NGC_MLP}
_DTYPES = {"f32": NGC_F32, "bf16": NGC_BF16, "f64": NGC_F64}

_HERE = os.path.dirname(os.path.abspath(__file__))


def lib_path() -> str:
    return os.path.join(_HERE, "libngc.so")


class NgcError(RuntimeError):
    def __init__(self, status: int, what: str, cuda: int = 0):
        self.status = status
        self.cuda = cuda
        super().__init__(f"{what}: status {status}" + (f" (cudaError {cuda})" if cuda else ""))


class Model(C.Structure):
    """ngc_model_t."""
    _fields_ = [("kind", C.c_int32), ("x_dtype", C.c_int32), ("rows_per_partition", C.c_int32),
                ("d", C.c_int32), ("n_classes", C.c_int32), ("hidden", C.c_int32)]

    @classmethod
    def make(cls, kind: str, x_dtype: str, rows: int, d: int, n_classes: int = 0, hidden: int = 0) -> "Model":
        return cls(_KINDS[kind], _DTYPES[x_dtype], rows, d, n_classes, hidden)


class StepInfo(C.Structure):
    """ngc_step_info_t."""
    _fields_ = [("layer", C.c_int32), ("sigma", C.c_int32), ("nS", C.c_int32), ("S", C.c_int32 * NGC_MAX_N),
                ("latency", C.c_double), ("tasks_done", C.c_int32 * NGC_MAX_N)]

    def responsive(self) -> np.ndarray:
        return np.array(self.S[: self.nS], dtype=np.int32)


_lib = None


def load_library() -> C.CDLL:
    """Loads libngc.so; raises if it is missing (there is no fallback path)."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise ImportError(f"{path} not found: build it with `python -m paper_2212_08580_b200.build`")
    lib = C.CDLL(path)
    vp, i32, i64, u64, dbl = C.c_void_p, C.c_int, C.c_int64, C.c_uint64, C.c_double
    P = C.POINTER
    sig = {
        "ngc_num_params": (i64, [P(Model)]),
        "ngc_plan": (i32, [i32, i32, P(C.c_int), i32, u64, dbl, dbl, P(vp)]),
        "ngc_plan_destroy": (None, [vp]),
        "ngc_plan_B": (i32, [vp, i32, P(P(dbl)), P(i32)]),
        "ngc_plan_schedule": (i32, [vp, P(P(C.c_int32)), P(P(C.c_int32))]),
        "ngc_set_coded_dtype": (i32, [vp, i32]),
        "ngc_coded_dtype": (i32, [vp, P(Model)]),
        "ngc_select": (i32, [vp, P(dbl), P(StepInfo)]),
        "ngc_prepare_data": (i32, [vp, P(Model), vp, vp]),
        "ngc_shard_prepare_data": (i32, [vp, P(Model), vp, i32, vp]),
        "ngc_shard_gradients": (i32, [vp, P(Model), vp, vp, vp, i32, vp, i64, vp]),
        "ngc_shard_encode_decode": (i32, [vp, P(Model), i32, i32, i32, vp, i64, P(C.c_int32), i32, vp, vp, vp]),
        "ngc_grad_encode": (i32, [vp, P(Model), vp, vp, vp, i32, vp, vp]),
        "ngc_grad_encode_static": (i32, [vp, P(Model), vp, vp, vp, i32, vp, vp, vp]),
        "ngc_decode_vector": (i32, [vp, i32, P(C.c_int32), i32, P(dbl)]),
        "ngc_decode_vectors": (i32, [vp, i32, P(C.c_int32), i32, i32, P(dbl), P(dbl)]),
        "ngc_decode": (i32, [vp, i32, P(C.c_int32), i32, vp, i32, i64, vp, vp]),
        "ngc_step": (i32, [vp, P(Model), vp, vp, vp, P(dbl), vp, vp, P(StepInfo), vp]),
        "ngc_step_host": (i32, [vp, P(Model), vp, vp, vp, P(dbl), vp, P(StepInfo)]),
        "ngc_latency_cdf_gc": (dbl, [i32, i32, dbl, dbl, dbl, dbl, dbl, dbl]),
        "ngc_latency_cdf_ngc": (dbl, [i32, i32, dbl, dbl, dbl, dbl, dbl, dbl]),
        "ngc_latency_mc": (i32, [vp, u64, i64, dbl, dbl, dbl, vp, vp, vp]),
        "ngc_gd_update": (i32, [vp, vp, i64, C.c_float, vp]),
        "ngc_sample_times": (i32, [u64, i32, i32, dbl, dbl, dbl, P(dbl)]),
        "ngc_selftest_wait_timeout": (i32, [vp, i64, vp]),
        "ngc_dense_schedule": (i32, [i32, i32, i32, i32, i32, vp, i32, P(i32), P(i32)]),
        "ngc_profile_enable": (i32, [vp, i32]),
        "ngc_profile_read": (i32, [vp, P(dbl), P(i64)]),
        "ngc_workspace_bytes": (C.c_size_t, [vp]),
        "ngc_device_status": (i32, [vp, P(dbl)]),
        "ngc_last_cuda_error": (i32, [vp]),
        "ngc_launch_count": (i64, [vp]),
        "ngc_strerror": (C.c_char_p, [i32]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


def _dptr(a) -> C.POINTER(C.c_double):
    return a.ctypes.data_as(C.POINTER(C.c_double))


def _iptr(a) -> C.POINTER(C.c_int32):
    return a.ctypes.data_as(C.POINTER(C.c_int32))


def _addr(t) -> int:
    """Address of a torch tensor's storage (device or host) or of a numpy array."""
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    return t.ctypes.data


def sample_times(seed: int, n: int, tasks: int, shift: float, rate: float, p_fail: float) -> np.ndarray:
    out = np.empty((n, tasks), dtype=np.float64)
    rc = load_library().ngc_sample_times(seed, n, tasks, shift, rate, p_fail, _dptr(out))
    if rc != 0:
        raise NgcError(rc, "ngc_sample_times")
    return out


def dense_schedule(batch: int, m_blocks: int, n_cols: int, k_chunks: int, max_pairs: int):
    """ngc_dense_schedule: (units [n][8] int32 = pair, round, partition, M block, c0, w0, c1, w1; number of pairs)."""
    lib = load_library()
    n_units, n_pairs = C.c_int32(0), C.c_int32(0)
    rc = lib.ngc_dense_schedule(batch, m_blocks, n_cols, k_chunks, max_pairs, None, 0, C.byref(n_units),
                                C.byref(n_pairs))
    if rc != 0:
        raise NgcError(rc, "ngc_dense_schedule")
    units = np.empty((n_units.value, 8), dtype=np.int32)
    rc = lib.ngc_dense_schedule(batch, m_blocks, n_cols, k_chunks, max_pairs, units.ctypes.data_as(C.c_void_p),
                                units.shape[0], C.byref(n_units), C.byref(n_pairs))
    if rc != 0:
        raise NgcError(rc, "ngc_dense_schedule")
    return units, n_pairs.value


def latency_cdf_gc(n, sigma, t, lam, rho, gamma, eps, p_fail) -> float:
    """Lemma 2: P(T_GC <= t)."""
    return float(load_library().ngc_latency_cdf_gc(n, sigma, t, lam, rho, gamma, eps, p_fail))


def latency_cdf_ngc(n, s_max, t, lam, rho, gamma, eps, p_fail) -> float:
    """Theorem 1: P(T_NGC <= t) of the fully nested code."""
    return float(load_library().ngc_latency_cdf_ngc(n, s_max, t, lam, rho, gamma, eps, p_fail))


def gd_update(theta, grad, step: float, stream: int = 0):
    """theta <- theta - step * grad on the device (Eq. 1 with step = eta / m)."""
    rc = load_library().ngc_gd_update(_addr(theta), _addr(grad), int(theta.numel()), float(step), stream)
    if rc != 0:
        raise NgcError(rc, "ngc_gd_update")


class Plan:
    """Owns an ngc_plan_t*.  Methods carry the names of the C entry points without the prefix."""

    def __init__(self, n_workers: int, levels, n_partitions: int | None = None, seed: int = 0,
                 gamma: float = 0.0, eps: float = 0.0):
        self._lib = load_library()
        self.n = int(n_workers)
        self.levels = [int(s) for s in levels]
        self.k = int(n_partitions if n_partitions is not None else n_workers)
        arr = (C.c_int * len(self.levels))(*self.levels)
        h = C.c_void_p()
        rc = self._lib.ngc_plan(self.n, len(self.levels), arr, self.k, seed, gamma, eps, C.byref(h))
        if rc != 0:
            raise NgcError(rc, "ngc_plan")
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            self._lib.ngc_plan_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int, what: str):
        if rc != 0:
            raise NgcError(rc, what + ": " + self._lib.ngc_strerror(rc).decode(),
                           self._lib.ngc_last_cuda_error(self._h))

    # ---- introspection
    def B(self, layer: int) -> np.ndarray:
        """Windowed coefficients, n x (s+1): row i = B[i, i..i+s mod n]."""
        ptr = C.POINTER(C.c_double)()
        w = C.c_int()
        self._check(self._lib.ngc_plan_B(self._h, layer, C.byref(ptr), C.byref(w)), "ngc_plan_B")
        return np.ctypeslib.as_array(ptr, shape=(self.n, w.value)).copy()

    def B_dense(self, layer: int) -> np.ndarray:
        Bw = self.B(layer)
        out = np.zeros((self.n, self.n))
        for i in range(self.n):
            for t in range(Bw.shape[1]):
                out[i, (i + t) % self.n] = Bw[i, t]
        return out

    def schedule(self):
        order = C.POINTER(C.c_int32)()
        tpl = C.POINTER(C.c_int32)()
        self._check(self._lib.ngc_plan_schedule(self._h, C.byref(order), C.byref(tpl)), "ngc_plan_schedule")
        return (np.ctypeslib.as_array(order, shape=(self.n, self.levels[-1] + 1)).copy(),
                np.ctypeslib.as_array(tpl, shape=(len(self.levels),)).copy())

    def set_coded_dtype(self, dtype: int):
        self._check(self._lib.ngc_set_coded_dtype(self._h, dtype), "ngc_set_coded_dtype")

    def coded_dtype(self, model: Model) -> int:
        return self._lib.ngc_coded_dtype(self._h, C.byref(model))

    def num_params(self, model: Model) -> int:
        return int(self._lib.ngc_num_params(C.byref(model)))

    # ---- host-side rule
    def select(self, task_times: np.ndarray) -> StepInfo:
        t = np.ascontiguousarray(task_times, dtype=np.float64)
        assert t.shape == (self.n, self.levels[-1] + 1)
        info = StepInfo()
        self._check(self._lib.ngc_select(self._h, _dptr(t), C.byref(info)), "ngc_select")
        return info

    # ---- device path
    def prepare_data(self, model: Model, X, stream: int = 0):
        """ngc_prepare_data: what the library derives from the data matrix alone, made once (X=None drops it)."""
        self._check(self._lib.ngc_prepare_data(self._h, C.byref(model), _addr(X) if X is not None else None, stream),
                    "ngc_prepare_data")

    def shard_prepare_data(self, model: Model, X_local, n_local: int, stream: int = 0):
        """ngc_shard_prepare_data: prepare_data for a shard of n_local partition groups."""
        self._check(self._lib.ngc_shard_prepare_data(self._h, C.byref(model),
                                                     _addr(X_local) if X_local is not None else None, n_local, stream),
                    "ngc_shard_prepare_data")

    def shard_gradients(self, model: Model, theta, X_local, y_local, n_local: int, G, ld: int, stream: int = 0):
        self._check(self._lib.ngc_shard_gradients(self._h, C.byref(model), _addr(theta), _addr(X_local), _addr(y_local),
                                                  n_local, _addr(G), ld, stream), "ngc_shard_gradients")

    def shard_encode_decode(self, model: Model, layer: int, first_worker: int, n_local: int, G_window, ld: int, S,
                            coded, partial, stream: int = 0):
        S = np.ascontiguousarray(S, dtype=np.int32)
        self._check(self._lib.ngc_shard_encode_decode(self._h, C.byref(model), layer, first_worker, n_local,
                                                      _addr(G_window), ld, _iptr(S), len(S), _addr(coded),
                                                      _addr(partial), stream), "ngc_shard_encode_decode")

    def grad_encode(self, model: Model, theta, X, y, layer: int, coded, stream: int = 0):
        self._check(self._lib.ngc_grad_encode(self._h, C.byref(model), _addr(theta), _addr(X), _addr(y), layer,
                                              _addr(coded), stream), "ngc_grad_encode")

    def grad_encode_static(self, model: Model, theta, X, y, layer: int, coded, status=None, stream: int = 0):
        """ngc_grad_encode_static: same result as grad_encode, but no device memory is allocated
        (scratch comes from a fixed array inside the library; see include/ngc.h for the limit)."""
        self._check(self._lib.ngc_grad_encode_static(self._h, C.byref(model), _addr(theta), _addr(X), _addr(y), layer,
                                                     _addr(coded), _addr(status) if status is not None else None,
                                                     stream), "ngc_grad_encode_static")

    def decode_vector(self, layer: int, S) -> np.ndarray:
        S = np.ascontiguousarray(S, dtype=np.int32)
        a = np.empty(self.n, dtype=np.float64)
        self._check(self._lib.ngc_decode_vector(self._h, layer, _iptr(S), len(S), _dptr(a)), "ngc_decode_vector")
        return a

    def decode_vectors(self, layer: int, S_batch):
        S = np.ascontiguousarray(S_batch, dtype=np.int32)
        batch, nS = S.shape
        a = np.empty((batch, self.n), dtype=np.float64)
        res = np.empty(batch, dtype=np.float64)
        self._check(self._lib.ngc_decode_vectors(self._h, layer, _iptr(S), nS, batch, _dptr(a), _dptr(res)),
                    "ngc_decode_vectors")
        return a, res

    def decode(self, layer: int, S, coded, coded_dtype: int, n_params: int, grad, stream: int = 0):
        S = np.ascontiguousarray(S, dtype=np.int32)
        self._check(self._lib.ngc_decode(self._h, layer, _iptr(S), len(S), _addr(coded), coded_dtype, n_params,
                                         _addr(grad), stream), "ngc_decode")

    def step(self, model: Model, theta, X, y, task_times: np.ndarray, coded, grad, stream: int = 0) -> StepInfo:
        t = np.ascontiguousarray(task_times, dtype=np.float64)
        info = StepInfo()
        self._check(self._lib.ngc_step(self._h, C.byref(model), _addr(theta), _addr(X), _addr(y), _dptr(t),
                                       _addr(coded), _addr(grad), C.byref(info), stream), "ngc_step")
        return info

    def step_host(self, model: Model, theta, X, y, task_times: np.ndarray, grad) -> StepInfo:
        t = np.ascontiguousarray(task_times, dtype=np.float64)
        info = StepInfo()
        self._check(self._lib.ngc_step_host(self._h, C.byref(model), _addr(theta), _addr(X), _addr(y), _dptr(t),
                                            _addr(grad), C.byref(info)), "ngc_step_host")
        return info

    def latency_mc(self, seed: int, rho: float, lam: float, p_fail: float, latency, level, stream: int = 0):
        """Monte Carlo of the stopping rule: fills the device tensors latency (float64) and level (int32)."""
        self._check(self._lib.ngc_latency_mc(self._h, seed, int(latency.numel()), rho, lam, p_fail, _addr(latency),
                                             _addr(level), stream), "ngc_latency_mc")

    def device_status(self) -> float:
        res = C.c_double()
        self._check(self._lib.ngc_device_status(self._h, C.byref(res)), "ngc_device_status")
        return res.value

    def device_status_code(self) -> int:
        """Raw return value of ngc_device_status (0, NGC_ERR_TIMEOUT or NGC_ERR_SINGULAR)."""
        return int(self._lib.ngc_device_status(self._h, None))

    def selftest_wait_timeout(self, limit_cycles: int, stream: int = 0):
        self._check(self._lib.ngc_selftest_wait_timeout(self._h, int(limit_cycles), stream),
                    "ngc_selftest_wait_timeout")

    def profile_enable(self, on: bool):
        self._check(self._lib.ngc_profile_enable(self._h, int(on)), "ngc_profile_enable")

    def profile_read(self):
        """(summed milliseconds of the bracketed fused-gradient kernels, their count) since the last read."""
        ms, cnt = C.c_double(), C.c_int64()
        self._check(self._lib.ngc_profile_read(self._h, C.byref(ms), C.byref(cnt)), "ngc_profile_read")
        return ms.value, cnt.value

    def workspace_bytes(self) -> int:
        return int(self._lib.ngc_workspace_bytes(self._h))

    def launch_count(self) -> int:
        return int(self._lib.ngc_launch_count(self._h))
