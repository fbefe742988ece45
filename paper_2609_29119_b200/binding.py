"""ctypes binding with the same names as include/cqt.h.

Argument marshalling only: every step of the transform runs in the CUDA kernels of
libcqt_b200.so.  torch is used for device memory and streams.  There is no CPU fallback:
if the library is missing, load_library() raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

WIN_HANN, WIN_BLACKMAN_HARRIS = 0, 1
M_MULT4, M_SMOOTH, M_POW2 = 0, 1, 2

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB: Optional[C.CDLL] = None


class CqtError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: status {status} ({status_string(status)})")
        self.status = status


class PlanDesc(C.Structure):
    _fields_ = [("fs", C.c_double), ("fmin", C.c_double), ("fmax", C.c_double), ("bins_per_octave", C.c_int),
                ("L", C.c_int64), ("window", C.c_int), ("m_policy", C.c_int), ("min_win", C.c_double),
                ("device", C.c_int)]


class PlanTuning(C.Structure):
    _fields_ = [("max_cta_elems", C.c_int64), ("two_pass_min", C.c_int64)]


class BandListDesc(C.Structure):
    _fields_ = [("fs", C.c_double), ("L", C.c_int64), ("window", C.c_int), ("m_policy", C.c_int), ("device", C.c_int),
                ("n_bands", C.c_int64), ("centre_hz", C.POINTER(C.c_double)), ("width_bins", C.POINTER(C.c_double)),
                ("group", C.POINTER(C.c_int32))]


class BandInfo(C.Structure):
    _fields_ = [("centre_hz", C.c_double), ("centre_bin", C.c_int64), ("support", C.c_int64),
                ("first_offset", C.c_int64), ("M", C.c_int64), ("coeff_offset", C.c_int64),
                ("table_offset", C.c_int64), ("is_sideband", C.c_int), ("launch_class", C.c_int)]


EXPORTS = {
    "cqt_plan_create": (C.c_int, [C.c_double, C.c_double, C.c_double, C.c_int, C.c_int64, C.c_int, C.POINTER(C.c_void_p)]),
    "cqt_plan_create_ex": (C.c_int, [C.POINTER(PlanDesc), C.POINTER(C.c_void_p)]),
    "cqt_plan_create_tuned": (C.c_int, [C.POINTER(PlanDesc), C.POINTER(PlanTuning), C.POINTER(C.c_void_p)]),
    "cqt_plan_create_bands": (C.c_int, [C.POINTER(BandListDesc), C.POINTER(C.c_void_p)]),
    "cqt_multires_bands": (C.c_int, [C.c_double, C.c_double, C.c_int64, C.POINTER(C.c_int), C.POINTER(C.c_int), C.c_int,
                                     C.c_double, C.c_int64, C.POINTER(C.c_double), C.POINTER(C.c_double),
                                     C.POINTER(C.c_int32), C.POINTER(C.c_int64)]),
    "cqt_plan_destroy": (C.c_int, [C.c_void_p]),
    "cqt_plan_num_bands": (C.c_int64, [C.c_void_p]),
    "cqt_plan_coeff_count": (C.c_int64, [C.c_void_p]),
    "cqt_plan_signal_length": (C.c_int64, [C.c_void_p]),
    "cqt_plan_table_length": (C.c_int64, [C.c_void_p]),
    "cqt_plan_device": (C.c_int, [C.c_void_p]),
    "cqt_static_workspace_bytes": (C.c_size_t, []),
    "cqt_analyse_static_ws": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p]),
    "cqt_plan_band_info": (C.c_int, [C.c_void_p, C.c_int64, C.POINTER(BandInfo)]),
    "cqt_plan_workspace_bytes": (C.c_size_t, [C.c_void_p, C.c_int64]),
    "cqt_plan_tables": (C.c_int, [C.c_void_p, C.POINTER(C.POINTER(C.c_float)), C.POINTER(C.POINTER(C.c_float))]),
    "cqt_plan_check": (C.c_int, [C.c_void_p]),
    "cqt_plan_launch_count": (C.c_int64, [C.c_void_p]),
    "cqt_plan_set_timing": (C.c_int, [C.c_void_p, C.c_int]),
    "cqt_plan_read_timing": (C.c_int, [C.c_void_p, C.POINTER(C.c_char_p), C.POINTER(C.c_float), C.c_int64, C.POINTER(C.c_int64)]),
    "cqt_analyse": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "cqt_synthesise": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_size_t, C.c_void_p]),
    "cqt_analyse_adjoint": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_size_t, C.c_void_p]),
    "cqt_synthesise_adjoint": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "slicq_create": (C.c_int, [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.POINTER(C.c_void_p)]),
    "slicq_push": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.POINTER(C.c_int64)]),
    "slicq_coeffs": (C.c_int, [C.c_void_p, C.c_int64, C.POINTER(C.c_void_p)]),
    "slicq_pull": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.POINTER(C.c_int64)]),
    "slicq_flush": (C.c_int, [C.c_void_p, C.c_void_p]),
    "slicq_reset": (C.c_int, [C.c_void_p]),
    "slicq_destroy": (C.c_int, [C.c_void_p]),
    "slicq_assembled_length": (C.c_int64, [C.c_void_p, C.c_int64]),
    "slicq_assemble": (C.c_int, [C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p]),
    "slicq_state_bytes": (C.c_size_t, [C.c_void_p]),
    "slicq_save_state": (C.c_int, [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "slicq_load_state": (C.c_int, [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "slicq_device_bytes": (C.c_size_t, [C.c_void_p]),
    "cqt_status_string": (C.c_char_p, [C.c_int]),
}


def lib_path() -> str:
    return os.path.join(_HERE, "libcqt_b200.so")


def load_library() -> C.CDLL:
    global _LIB
    if _LIB is None:
        path = lib_path()
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: build it with `python -m paper_2609_29119_b200.build` "
                               "(there is no CPU fallback)")
        lib = C.CDLL(path)
        for name, (res, args) in EXPORTS.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _LIB = lib
    return _LIB


def status_string(status: int) -> str:
    return load_library().cqt_status_string(status).decode()


def _check(status: int, what: str) -> None:
    if status != 0:
        raise CqtError(status, what)


def multires_bands(fs: float, fmin: float, L: int, sections, min_win: float = 4.0):
    """cqt_multires_bands: (centre_hz, width_bins, octave) lists for sections of (octaves, bins per octave)."""
    lib = load_library()
    ns = len(sections)
    octs = (C.c_int * ns)(*[int(s[0]) for s in sections])
    bpo = (C.c_int * ns)(*[int(s[1]) for s in sections])
    n = C.c_int64(0)
    _check(lib.cqt_multires_bands(fs, fmin, L, octs, bpo, ns, min_win, 0, None, None, None, C.byref(n)), "cqt_multires_bands")
    c, w, g = (C.c_double * n.value)(), (C.c_double * n.value)(), (C.c_int32 * n.value)()
    _check(lib.cqt_multires_bands(fs, fmin, L, octs, bpo, ns, min_win, n.value, c, w, g, C.byref(n)), "cqt_multires_bands")
    return list(c), list(w), list(g)


def _stream_ptr(stream) -> int:
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


class Plan:
    """cqt_plan_create_ex / cqt_plan_destroy plus the four transforms on torch CUDA tensors."""

    def __init__(self, fs: float, fmin: float, fmax: float, bins_per_octave: int, L: int, window: int = WIN_HANN,
                 m_policy: int = M_MULT4, min_win: float = 4.0, device: Optional[int] = None,
                 max_cta_elems: int = 0, two_pass_min: int = 0):
        """max_cta_elems, two_pass_min: the fields of cqt_plan_tuning (0 = default); either of them non-zero
        creates the plan with cqt_plan_create_tuned."""
        self.lib = load_library()
        if device is None:
            import torch
            device = torch.cuda.current_device()
        desc = PlanDesc(fs, fmin, fmax, bins_per_octave, L, window, m_policy, min_win, device)
        h = C.c_void_p()
        if max_cta_elems or two_pass_min:
            tune = PlanTuning(max_cta_elems, two_pass_min)
            _check(self.lib.cqt_plan_create_tuned(C.byref(desc), C.byref(tune), C.byref(h)), "cqt_plan_create_tuned")
        else:
            _check(self.lib.cqt_plan_create_ex(C.byref(desc), C.byref(h)), "cqt_plan_create_ex")
        self._adopt(h, device)

    @classmethod
    def from_bands(cls, fs: float, L: int, centre_hz, width_bins, group=None, window: int = WIN_HANN,
                   m_policy: int = M_MULT4, device: Optional[int] = None) -> "Plan":
        """cqt_plan_create_bands: a plan from an explicit list of regular bands."""
        self = cls.__new__(cls)
        self.lib = load_library()
        if device is None:
            import torch
            device = torch.cuda.current_device()
        n = len(centre_hz)
        if len(width_bins) != n or (group is not None and len(group) != n):
            raise ValueError("need one width (and one group) per band centre")
        c = (C.c_double * n)(*[float(v) for v in centre_hz])
        w = (C.c_double * n)(*[float(v) for v in width_bins])
        g = (C.c_int32 * n)(*[int(v) for v in group]) if group is not None else None
        desc = BandListDesc(fs, L, window, m_policy, device, n, c, w, g)
        h = C.c_void_p()
        _check(self.lib.cqt_plan_create_bands(C.byref(desc), C.byref(h)), "cqt_plan_create_bands")
        self._adopt(h, device)
        return self

    def _adopt(self, h, device) -> None:
        self.handle = h
        self.device = device
        self.N = int(self.lib.cqt_plan_signal_length(h))
        self.num_bands = int(self.lib.cqt_plan_num_bands(h))
        self.coeff_count = int(self.lib.cqt_plan_coeff_count(h))
        self.table_length = int(self.lib.cqt_plan_table_length(h))
        self._ws = None

    def close(self) -> None:
        if getattr(self, "handle", None):
            self.lib.cqt_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- queries
    def band_info(self, band: int) -> BandInfo:
        bi = BandInfo()
        _check(self.lib.cqt_plan_band_info(self.handle, band, C.byref(bi)), "cqt_plan_band_info")
        return bi

    def bands(self):
        return [self.band_info(i) for i in range(self.num_bands)]

    def tables(self):
        import numpy as np
        g, h = C.POINTER(C.c_float)(), C.POINTER(C.c_float)()
        _check(self.lib.cqt_plan_tables(self.handle, C.byref(g), C.byref(h)), "cqt_plan_tables")
        n = self.table_length
        return (np.ctypeslib.as_array(g, shape=(n,)).copy(), np.ctypeslib.as_array(h, shape=(n,)).copy())

    def workspace_bytes(self, batch: int) -> int:
        return int(self.lib.cqt_plan_workspace_bytes(self.handle, batch))

    def workspace(self, batch: int):
        import torch
        need = self.workspace_bytes(batch)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=f"cuda:{self.device}")
        return self._ws

    def check(self) -> int:
        """cqt_plan_check: 0, or -7 if a debug-bounds build recorded an out-of-range index (printed to stderr)."""
        return int(self.lib.cqt_plan_check(self.handle))

    def launch_count(self) -> int:
        return int(self.lib.cqt_plan_launch_count(self.handle))

    def set_timing(self, enable: bool) -> None:
        _check(self.lib.cqt_plan_set_timing(self.handle, 1 if enable else 0), "cqt_plan_set_timing")

    def read_timing(self, capacity: int = 4096):
        """[(kernel name, milliseconds)] for every kernel launched since the last read (synchronises)."""
        names = (C.c_char_p * capacity)()
        ms = (C.c_float * capacity)()
        n = C.c_int64()
        _check(self.lib.cqt_plan_read_timing(self.handle, names, ms, capacity, C.byref(n)), "cqt_plan_read_timing")
        m = min(int(n.value), capacity)
        return [(names[i].decode(), float(ms[i])) for i in range(m)]

    # ---- transforms (x: [batch, >= valid_len] float32 cuda; c: [batch, coeff_count] complex64 cuda)
    def _sig(self, x, valid_len):
        import torch
        assert x.is_cuda and x.dtype == torch.float32 and x.dim() == 2 and x.stride(1) == 1
        return x.shape[0], (x.shape[1] if valid_len is None else valid_len), x.stride(0)

    def analyse(self, x, valid_len=None, out=None, ws=None, stream=None, _fn="cqt_analyse"):
        import torch
        batch, vl, stride = self._sig(x, valid_len)
        if out is None:
            out = torch.empty((batch, self.coeff_count), dtype=torch.complex64, device=x.device)
        ws = self.workspace(batch) if ws is None else ws
        _check(getattr(self.lib, _fn)(self.handle, x.data_ptr(), stride, batch, vl, out.data_ptr(), ws.data_ptr(),
                                      ws.numel(), _stream_ptr(stream)), _fn)
        return out

    def analyse_static_ws(self, x, valid_len=None, out=None, stream=None):
        """cqt_analyse_static_ws: analysis for callers that cannot allocate; scratch is the library's own
        fixed 16 MiB array (shared by all calls, so overlapping calls race), limited batch."""
        import torch
        batch, vl, stride = self._sig(x, valid_len)
        if out is None:
            out = torch.empty((batch, self.coeff_count), dtype=torch.complex64, device=x.device)
        _check(self.lib.cqt_analyse_static_ws(self.handle, x.data_ptr(), stride, batch, vl, out.data_ptr(),
                                              _stream_ptr(stream)), "cqt_analyse_static_ws")
        return out

    def synthesise(self, c, valid_len=None, out=None, ws=None, stream=None, _fn="cqt_synthesise"):
        import torch
        assert c.is_cuda and c.dtype == torch.complex64 and c.dim() == 2 and c.is_contiguous()
        assert c.shape[1] == self.coeff_count
        batch = c.shape[0]
        vl = self.N if valid_len is None else valid_len
        if out is None:
            out = torch.empty((batch, vl), dtype=torch.float32, device=c.device)
        ws = self.workspace(batch) if ws is None else ws
        _check(getattr(self.lib, _fn)(self.handle, c.data_ptr(), batch, vl, out.data_ptr(), out.stride(0), ws.data_ptr(),
                                      ws.numel(), _stream_ptr(stream)), _fn)
        return out

    def analyse_adjoint(self, c_bar, valid_len=None, out=None, ws=None, stream=None):
        return self.synthesise(c_bar, valid_len, out, ws, stream, _fn="cqt_analyse_adjoint")

    def synthesise_adjoint(self, x_bar, valid_len=None, out=None, ws=None, stream=None):
        return self.analyse(x_bar, valid_len, out, ws, stream, _fn="cqt_synthesise_adjoint")


class SliCQ:
    """slicq_create / push / pull / flush on torch CUDA tensors ([channels, n] float32)."""

    def __init__(self, plan: Plan, channels: int, transition: int, max_slices_in_flight: int):
        self.plan, self.lib, self.channels = plan, plan.lib, channels
        h = C.c_void_p()
        _check(self.lib.slicq_create(plan.handle, channels, transition, max_slices_in_flight, C.byref(h)), "slicq_create")
        self.handle = h

    def close(self):
        if getattr(self, "handle", None):
            self.lib.slicq_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def device_bytes(self) -> int:
        return int(self.lib.slicq_device_bytes(self.handle))

    def push(self, x, stream=None) -> int:
        done = C.c_int64()
        n = x.shape[1]
        _check(self.lib.slicq_push(self.handle, x.data_ptr() if n else None, x.stride(0) if n else 0, n,
                                   _stream_ptr(stream), C.byref(done)), "slicq_push")
        return int(done.value)

    def coeffs(self, slice_index: int):
        """complex64 view [channels, coeff_count] of one analysed slice (valid until it is pulled)."""
        import torch
        p = C.c_void_p()
        _check(self.lib.slicq_coeffs(self.handle, slice_index, C.byref(p)), "slicq_coeffs")
        return _DevicePtrTensor(p.value, (self.channels, self.plan.coeff_count), self.plan.device)

    def pull(self, y, stream=None) -> int:
        wrote = C.c_int64()
        _check(self.lib.slicq_pull(self.handle, y.data_ptr(), y.stride(0), y.shape[1], _stream_ptr(stream),
                                   C.byref(wrote)), "slicq_pull")
        return int(wrote.value)

    def flush(self, stream=None) -> None:
        _check(self.lib.slicq_flush(self.handle, _stream_ptr(stream)), "slicq_flush")

    def reset(self) -> None:
        _check(self.lib.slicq_reset(self.handle), "slicq_reset")

    def assemble(self, first_slice: int, n_slices: int, out=None, stream=None):
        """slicq_assemble: [channels, (n_slices + 1) * coeff_count / 2] complex64, one time series per band."""
        import torch
        n = int(self.lib.slicq_assembled_length(self.handle, n_slices))
        if out is None:
            out = torch.empty((self.channels, n), dtype=torch.complex64, device=f"cuda:{self.plan.device}")
        _check(self.lib.slicq_assemble(self.handle, first_slice, n_slices, out.data_ptr(), out.stride(0),
                                       _stream_ptr(stream)), "slicq_assemble")
        return out

    def save_state(self, stream=None) -> bytes:
        n = int(self.lib.slicq_state_bytes(self.handle))
        buf = C.create_string_buffer(n)
        _check(self.lib.slicq_save_state(self.handle, buf, n, _stream_ptr(stream)), "slicq_save_state")
        return buf.raw

    def load_state(self, state: bytes, stream=None) -> None:
        buf = C.create_string_buffer(state, len(state))
        _check(self.lib.slicq_load_state(self.handle, buf, len(state), _stream_ptr(stream)), "slicq_load_state")


class _DeviceArray:
    """Exposes a device buffer owned by the library through the CUDA array interface."""

    def __init__(self, ptr: int, shape):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": "<c8", "data": (ptr, False), "version": 3,
                                         "strides": None}


def _DevicePtrTensor(ptr: int, shape, device: int):
    """Zero-copy complex64 torch view of a device buffer owned by the library."""
    import torch
    return torch.as_tensor(_DeviceArray(ptr, shape), device=f"cuda:{device}")
