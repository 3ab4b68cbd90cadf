"""ctypes binding of libdraco.so: argument marshalling only.

Every function takes raw device pointers (``tensor.data_ptr()``) or torch
tensors and a CUDA stream handle; PyTorch is used by callers for device memory
and streams, never for arithmetic on the path.
"""
from __future__ import annotations

import ctypes as C
import os

REP, CYC, CYC_PACKED = 0, 1, 2
ADV_REVGRAD, ADV_CONST, ADV_GAUSS = 0, 1, 2
OK, EINVAL, ECUDA, ETOOMANY, ENOMEM, EINTERNAL, ELIMIT, ENOMAJ, EUNSURE = 0, -1, -2, -3, -4, -5, -6, 1, 2
MAX_N = 128

_PKG = os.path.dirname(os.path.abspath(__file__))


class DracoError(RuntimeError):
    pass


class DracoInfo(C.Structure):
    _fields_ = [("status", C.c_int32), ("n_flagged", C.c_int32), ("locator_rank", C.c_int32),
                ("n_active", C.c_int32), ("no_majority", C.c_uint64), ("scale", C.c_double),
                ("max_syndrome", C.c_double), ("internal_error", C.c_int32), ("svd_sweeps", C.c_int32),
                ("locator_margin", C.c_double), ("im_residual", C.c_double), ("re_max", C.c_double)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


def library_path() -> str:
    return os.path.join(_PKG, "libdraco.so")


def _load() -> C.CDLL:
    path = library_path()
    if not os.path.exists(path):
        raise DracoError(f"{path} is missing: build it with `python -m paper_1803_09877_b200.build` "
                         "(there is no CPU fallback)")
    return C.CDLL(path)


lib = _load()

_vp, _i, _i64, _u64, _f = C.c_void_p, C.c_int, C.c_int64, C.c_uint64, C.c_float
_SIGS = {
    "draco_plan_create": ([_i, _i, _i64, _i, C.POINTER(_vp)], _i),
    "draco_plan_destroy": ([_vp], _i),
    "draco_plan_set_theta": ([_vp, C.c_double], _i),
    "draco_num_groups": ([_vp], _i),
    "draco_groups": ([_vp, C.POINTER(_i), C.POINTER(_i)], _i),
    "draco_cyc_W": ([_vp, C.POINTER(C.c_double)], _i),
    "draco_encode": ([_vp, _vp, _vp, _vp], _i),
    "draco_locate": ([_vp, _vp, _vp, _vp, _vp], _i),
    "draco_decode": ([_vp, _vp, _vp, _vp, _vp], _i),
    "draco_locate_decode": ([_vp, _vp, _vp, _vp, _vp, _vp], _i),
    "draco_decode_update": ([_vp, _vp, _vp, _vp, _f, _vp], _i),
    "draco_rep_vote": ([_vp, _vp, _vp, _vp, _vp, _vp], _i),
    "draco_cyc_project": ([_vp, _vp, _vp, _vp, _vp], _i),
    "draco_cyc_locate_from_projection": ([_vp, _vp, _vp, _vp], _i),
    "draco_cyc_project_noalloc": ([_i, _i64, _vp, _vp, _vp, _vp], _i),
    "draco_cyc_decode_vector": ([_vp, C.POINTER(C.c_double), _vp], _i),
    "draco_get_info": ([_vp, C.POINTER(DracoInfo), _vp], _i),
    "draco_pipeline_host": ([_vp, _vp, _vp, C.POINTER(_i), C.POINTER(_i), C.POINTER(_f), _i, _u64, _vp, _vp, _vp,
                             C.POINTER(DracoInfo)], _i),
    "draco_generate": ([_vp, _i, _i64, _i, _f, _f, _u64, _vp], _i),
    "draco_corrupt": ([_vp, _vp, C.POINTER(_i), C.POINTER(_i), C.POINTER(_f), _i, _u64, _vp], _i),
    "draco_strerror": ([_i], C.c_char_p),
    "draco_last_cuda_error": ([], C.c_char_p),
}
for _name, (_args, _res) in _SIGS.items():
    _fn = getattr(lib, _name)
    _fn.argtypes = _args
    _fn.restype = _res

EXPORTS = tuple(_SIGS)


def _check(rc: int) -> int:
    if rc < 0:
        msg = lib.draco_strerror(rc).decode()
        if rc == ECUDA:
            msg += ": " + lib.draco_last_cuda_error().decode()
        raise DracoError(f"libdraco: {msg} ({rc})")
    return rc


def _ptr(x):
    """Device / host address of a torch tensor, an int address, or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return x.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _adv_arrays(adv_idx, adv_model, adv_param):
    k = len(adv_idx)
    return ((_i * k)(*[int(a) for a in adv_idx]), (_i * k)(*[int(a) for a in adv_model]),
            (_f * k)(*[float(a) for a in adv_param]), k)


def cyc_project_noalloc(n: int, d: int, R, f, e, stream=None):
    """draco_cyc_project_noalloc: e = f R with the library's built-in scratch; needs no plan and allocates nothing."""
    return _check(lib.draco_cyc_project_noalloc(n, d, _ptr(R), _ptr(f), _ptr(e), _stream(stream)))


def generate(out, rows: int, length: int, row0: int = 0, mean: float = 0.0, std: float = 1.0, seed: int = 0,
             stream=None):
    """draco_generate: fill device [rows][length] fp32 with the seeded generator."""
    _check(lib.draco_generate(_ptr(out), rows, length, row0, mean, std, seed & 0xFFFFFFFFFFFFFFFF, _stream(stream)))


class Plan:
    """draco_plan: tables and scratch for one (n, s, d, code) on the current device."""

    def __init__(self, n: int, s: int, d: int, code: int):
        self.n, self.s, self.d, self.code = n, s, d, code
        h = _vp()
        _check(lib.draco_plan_create(n, s, d, code, C.byref(h)))
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            lib.draco_plan_destroy(self._h)
            self._h = None

    __del__ = close

    def set_theta(self, theta: float):
        _check(lib.draco_plan_set_theta(self._h, theta))

    def groups(self):
        g = _check(lib.draco_num_groups(self._h))
        first, size = (_i * max(g, 1))(), (_i * max(g, 1))()
        if g:
            _check(lib.draco_groups(self._h, first, size))
        return [(first[k], size[k]) for k in range(g)]

    def cyc_W(self):
        import numpy as np
        buf = (C.c_double * (2 * self.n * self.n))()
        _check(lib.draco_cyc_W(self._h, buf))
        a = np.frombuffer(buf, dtype=np.float64).reshape(self.n, self.n, 2)
        return a[..., 0] + 1j * a[..., 1]

    def encode(self, G, Z, stream=None):
        return _check(lib.draco_encode(self._h, _ptr(G), _ptr(Z), _stream(stream)))

    def locate(self, R, f, flags, stream=None):
        return _check(lib.draco_locate(self._h, _ptr(R), _ptr(f), _ptr(flags), _stream(stream)))

    def decode(self, R, flags, u, stream=None):
        return _check(lib.draco_decode(self._h, _ptr(R), _ptr(flags), _ptr(u), _stream(stream)))

    def decode_update(self, R, flags, w, scale: float, stream=None):
        return _check(lib.draco_decode_update(self._h, _ptr(R), _ptr(flags), _ptr(w), scale, _stream(stream)))

    def locate_decode(self, R, f, flags, u, stream=None):
        return _check(lib.draco_locate_decode(self._h, _ptr(R), _ptr(f), _ptr(flags), _ptr(u), _stream(stream)))

    def rep_vote(self, R, u=None, maj=None, flags=None, stream=None):
        return _check(lib.draco_rep_vote(self._h, _ptr(R), _ptr(u), _ptr(maj), _ptr(flags), _stream(stream)))

    def cyc_project(self, R, f, e, stream=None):
        return _check(lib.draco_cyc_project(self._h, _ptr(R), _ptr(f), _ptr(e), _stream(stream)))

    def cyc_locate_from_projection(self, e, flags, stream=None):
        return _check(lib.draco_cyc_locate_from_projection(self._h, _ptr(e), _ptr(flags), _stream(stream)))

    def cyc_decode_vector(self, stream=None):
        import numpy as np
        buf = (C.c_double * (2 * self.n))()
        _check(lib.draco_cyc_decode_vector(self._h, buf, _stream(stream)))
        a = np.frombuffer(buf, dtype=np.float64).reshape(self.n, 2)
        return a[:, 0] + 1j * a[:, 1]

    def info(self, stream=None) -> dict:
        out = DracoInfo()
        _check(lib.draco_get_info(self._h, C.byref(out), _stream(stream)))
        return out.as_dict()

    def corrupt(self, R, adv_idx, adv_model, adv_param, seed: int = 0, stream=None):
        idx, model, param, k = _adv_arrays(adv_idx, adv_model, adv_param)
        return _check(lib.draco_corrupt(self._h, _ptr(R), idx, model, param, k, seed & 0xFFFFFFFFFFFFFFFF,
                                        _stream(stream)))

    def pipeline_host(self, G_host, f_host, adv_idx, adv_model, adv_param, adv_seed, Z, u_host, flags_host) -> dict:
        idx, model, param, k = _adv_arrays(adv_idx, adv_model, adv_param)
        out = DracoInfo()
        _check(lib.draco_pipeline_host(self._h, _ptr(G_host), _ptr(f_host), idx, model, param, k,
                                       adv_seed & 0xFFFFFFFFFFFFFFFF, _ptr(Z), _ptr(u_host), _ptr(flags_host),
                                       C.byref(out)))
        return out.as_dict()
