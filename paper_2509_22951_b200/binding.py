"""ctypes binding of libtq.so: argument marshalling only, same names as include/tq.h.

Host arrays are numpy arrays; device memory is torch CUDA tensors (PyTorch is used for
device memory and streams only).  There is no CPU fallback: if libtq.so cannot be loaded (or
built with nvcc) importing this module raises.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass

import numpy as np
import torch

from . import build as _build

TQ_OK = 0
TQ_ERR_INVALID_ARG = -1
TQ_ERR_CORRUPT_STREAM = -2
TQ_ERR_BUFFER_TOO_SMALL = -3
TQ_ERR_UNSUPPORTED_SHAPE = -4
TQ_ERR_CUDA = -5
TQ_ERR_TIMEOUT = -6
TQ_ERR_NOMEM = -7
TQ_LAYOUT_STREAM = 0
TQ_LAYOUT_PLANES = 1
TQ_LAYOUT_TILES = 2
TQ_TILES_TABLE_WORDS = 33024
TQ_TILES_MAX_COLS = 65536
TQ_STATUS_BAD_CODE = 1
TQ_STATUS_BAD_ROW = 2
TQ_STATUS_WAIT_EXPIRED = 4

EXPORTS = [
    "tq_strerror", "tq_last_cuda_error", "tq_set_num_threads", "tq_quantize_tensor", "tq_quantize_tensor_bits", "tq_quantize_rows",
    "tq_quantize_rows_device", "tq_build_dictionary", "tq_build_dictionary_device_size", "tq_build_dictionary_device", "tq_dict_from_entries", "tq_dict_entries",
    "tq_encode", "tq_dict_free", "tq_dict_upload_size", "tq_dict_upload", "tq_ddict_free",
    "tq_upload_size", "tq_upload", "tq_upload_device_size", "tq_upload_device", "tq_upload_device_rows", "tq_tiles_image_host", "tq_dmat_get_info", "tq_decompress", "tq_fused_gemv",
    "tq_fused_gemv_host", "tq_fused_gemv_host_static", "tq_fused_gemm", "tq_gemm_workspace_size",
    "tq_fused_gemm_ws", "tq_decode_bf16", "tq_gemm_bf16_ws", "tq_decode_bf16_stack", "tq_gemm_plan_size", "tq_gemm_plan_create", "tq_gemm_plan_run",
    "tq_gemm_plan_status", "tq_gemm_plan_free", "tq_stack_size", "tq_stack_plan_host", "tq_stack_create",
    "tq_fused_gemv_stack", "tq_fused_gemv_stack_host", "tq_stack_launches", "tq_test_withhold_table_chunk", "tq_decompress_stack", "tq_stack_free", "tq_device_status", "tq_dmat_free",
]


class TqError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str | None = None):
        self.status = status
        if detail is None:
            detail = _lib.tq_last_cuda_error().decode() if status == TQ_ERR_CUDA else ""
        super().__init__(f"{where}: {_lib.tq_strerror(status).decode()} ({status}) {detail}")


class _Info(C.Structure):
    _fields_ = [("rows", C.c_uint32), ("cols", C.c_uint32), ("K", C.c_uint32),
                ("layout", C.c_int32), ("levels_signed", C.c_int32),
                ("n_hits", C.c_uint64), ("n_miss", C.c_uint64), ("stream_bytes", C.c_uint64),
                ("payload_bytes", C.c_uint64), ("device_bytes", C.c_uint64), ("n_raw_words", C.c_uint64)]


def _load() -> C.CDLL:
    path = _build.build_library()  # raises if the library is missing and cannot be built
    lib = C.CDLL(str(path))
    vp, u8p, u16p, u32p, u64p = C.c_void_p, C.POINTER(C.c_uint8), C.POINTER(C.c_uint16), C.POINTER(C.c_uint32), C.POINTER(C.c_uint64)
    f32p = C.POINTER(C.c_float)
    sig = {
        "tq_strerror": (C.c_char_p, [C.c_int]),
        "tq_last_cuda_error": (C.c_char_p, []),
        "tq_set_num_threads": (C.c_int, [C.c_int]),
        "tq_quantize_tensor": (C.c_int, [f32p, C.c_uint64, u8p, f32p, f32p]),
        "tq_quantize_tensor_bits": (C.c_int, [f32p, C.c_uint64, C.c_int, u8p, f32p, f32p]),
        "tq_quantize_rows": (C.c_int, [f32p, C.c_uint32, C.c_uint32, C.POINTER(C.c_int8), f32p]),
        "tq_quantize_rows_device": (C.c_int, [vp, C.c_uint32, C.c_uint32, vp, vp, vp]),
        "tq_build_dictionary": (C.c_int, [C.POINTER(u8p), u64p, C.c_int, C.c_uint32, C.POINTER(vp)]),
        "tq_build_dictionary_device_size": (C.c_int, [u64p, C.c_int, u64p]),
        "tq_build_dictionary_device": (C.c_int, [C.POINTER(vp), u64p, C.c_int, C.c_uint32, vp, C.c_uint64, vp, C.POINTER(vp)]),
        "tq_dict_from_entries": (C.c_int, [u8p, C.c_uint32, C.POINTER(vp)]),
        "tq_dict_entries": (C.c_int, [vp, u32p, C.POINTER(u8p), C.POINTER(u64p)]),
        "tq_encode": (C.c_int, [vp, u8p, C.c_uint64, u16p, C.c_uint64, u64p, u64p, u64p]),
        "tq_dict_free": (None, [vp]),
        "tq_dict_upload_size": (C.c_int, [vp, u64p]),
        "tq_dict_upload": (C.c_int, [vp, vp, C.c_uint64, vp, C.POINTER(vp)]),
        "tq_ddict_free": (None, [vp]),
        "tq_upload_size": (C.c_int, [u16p, C.c_uint64, C.c_uint32, C.c_uint32, C.c_int, u64p]),
        "tq_upload": (C.c_int, [vp, u16p, C.c_uint64, C.c_uint32, C.c_uint32, f32p, f32p, C.c_int,
                                C.c_int, vp, C.c_uint64, vp, C.POINTER(vp)]),
        "tq_upload_device_size": (C.c_int, [C.c_uint32, C.c_uint32, u64p]),
        "tq_upload_device": (C.c_int, [vp, vp, C.c_uint32, C.c_uint32, vp, vp, C.c_int, vp, C.c_uint64, vp, C.POINTER(vp)]),
        "tq_upload_device_rows": (C.c_int, [vp, vp, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint32, vp, vp, C.c_int, vp, C.c_uint64, vp,
                                            C.POINTER(vp)]),
        "tq_tiles_image_host": (C.c_int, [vp, u16p, C.c_uint64, C.c_uint32, C.c_uint32, f32p, f32p, u8p,
                                          C.c_uint64, u64p, u64p, u32p]),
        "tq_dmat_get_info": (C.c_int, [vp, C.POINTER(_Info)]),
        "tq_decompress": (C.c_int, [vp, vp, vp]),
        "tq_fused_gemv": (C.c_int, [vp, vp, C.c_int, vp, vp]),
        "tq_fused_gemv_host": (C.c_int, [vp, vp, C.c_int, vp, vp, vp, vp]),
        "tq_fused_gemv_host_static": (C.c_int, [vp, vp, C.c_int, vp, vp]),
        "tq_fused_gemm": (C.c_int, [vp, vp, C.c_int, vp, vp]),
        "tq_gemm_workspace_size": (C.c_int, [vp, u64p]),
        "tq_fused_gemm_ws": (C.c_int, [vp, vp, C.c_int, vp, vp, C.c_uint64, vp]),
        "tq_decode_bf16": (C.c_int, [vp, vp, C.c_uint64, vp]),
        "tq_gemm_bf16_ws": (C.c_int, [vp, vp, C.c_int, vp, vp, vp]),
        "tq_decode_bf16_stack": (C.c_int, [vp, vp, vp]),
        "tq_gemm_plan_size": (C.c_int, [C.c_int, u64p]),
        "tq_gemm_plan_create": (C.c_int, [C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.c_int, C.c_int, vp,
                                          C.c_uint64, vp, C.POINTER(vp)]),
        "tq_gemm_plan_run": (C.c_int, [vp, vp]),
        "tq_gemm_plan_status": (C.c_int, [vp, vp, u32p]),
        "tq_gemm_plan_free": (None, [vp]),
        "tq_stack_size": (C.c_int, [C.POINTER(vp), C.c_int, C.c_int, u64p]),
        "tq_stack_plan_host": (C.c_int, [C.c_int, u32p, u32p, C.POINTER(u32p), C.c_uint32, u32p, C.c_uint32, u32p, u32p]),
        "tq_stack_create": (C.c_int, [C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.c_int, C.c_int, vp, C.c_uint64, vp,
                                      C.POINTER(vp)]),
        "tq_fused_gemv_stack": (C.c_int, [vp, vp]),
        "tq_fused_gemv_stack_host": (C.c_int, [vp, vp, vp, C.c_uint64, vp, vp, C.c_uint64, vp]),
        "tq_stack_launches": (C.c_int, [vp]),
        "tq_test_withhold_table_chunk": (None, [C.c_int]),
        "tq_decompress_stack": (C.c_int, [vp, vp, vp]),
        "tq_stack_free": (None, [vp]),
        "tq_device_status": (C.c_int, [vp, vp, u32p]),
        "tq_dmat_free": (None, [vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    return lib


_lib = _load()


def _check(status: int, where: str) -> None:
    if status != TQ_OK:
        raise TqError(status, where)


def _np_ptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(C.POINTER(ctype))


def _stream_ptr(stream=None) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def tq_set_num_threads(n: int) -> int:
    return _lib.tq_set_num_threads(n)


# ------------------------------------------------------------------------------ host
def tq_quantize_tensor(x: np.ndarray):
    x = np.ascontiguousarray(x, dtype=np.float32)
    q = np.empty(x.shape, dtype=np.uint8)
    s, z = C.c_float(), C.c_float()
    _check(_lib.tq_quantize_tensor(_np_ptr(x, C.c_float), x.size, _np_ptr(q, C.c_uint8), C.byref(s), C.byref(z)),
           "tq_quantize_tensor")
    return q, np.float32(s.value), np.float32(z.value)


def tq_quantize_tensor_bits(x: np.ndarray, bits: int):
    x = np.ascontiguousarray(x, dtype=np.float32)
    q = np.empty(x.shape, dtype=np.uint8)
    s, z = C.c_float(), C.c_float()
    _check(_lib.tq_quantize_tensor_bits(_np_ptr(x, C.c_float), x.size, int(bits), _np_ptr(q, C.c_uint8), C.byref(s),
                                        C.byref(z)), "tq_quantize_tensor_bits")
    return q, np.float32(s.value), np.float32(z.value)


def tq_quantize_rows(w: np.ndarray):
    w = np.ascontiguousarray(w, dtype=np.float32)
    rows, cols = w.shape
    q = np.empty((rows, cols), dtype=np.int8)
    s = np.empty(rows, dtype=np.float32)
    _check(_lib.tq_quantize_rows(_np_ptr(w, C.c_float), rows, cols, _np_ptr(q, C.c_int8), _np_ptr(s, C.c_float)),
           "tq_quantize_rows")
    return q, s


def tq_quantize_rows_device(w: torch.Tensor, stream=None):
    assert w.is_cuda and w.dtype == torch.float32 and w.is_contiguous() and w.dim() == 2
    rows, cols = w.shape
    q = torch.empty((rows, cols), dtype=torch.int8, device=w.device)
    s = torch.empty(rows, dtype=torch.float32, device=w.device)
    _check(_lib.tq_quantize_rows_device(w.data_ptr(), rows, cols, q.data_ptr(), s.data_ptr(), _stream_ptr(stream)),
           "tq_quantize_rows_device")
    return q, s


class Dict:
    """Owner of a host tq_dict handle."""

    def __init__(self, handle: int):
        self._h = C.c_void_p(handle)

    def __del__(self):
        if getattr(self, "_h", None) and _lib is not None:
            _lib.tq_dict_free(self._h)
            self._h = None

    def _borrow(self):
        K, e, c = C.c_uint32(), C.POINTER(C.c_uint8)(), C.POINTER(C.c_uint64)()
        _check(_lib.tq_dict_entries(self._h, C.byref(K), C.byref(e), C.byref(c)), "tq_dict_entries")
        return K.value, e, c

    @property
    def K(self) -> int:
        return self._borrow()[0]

    @property
    def entries(self) -> np.ndarray:
        K, e, _ = self._borrow()
        return np.ctypeslib.as_array(e, shape=(K, 4)).copy() if K else np.zeros((0, 4), np.uint8)

    @property
    def counts(self) -> np.ndarray:
        K, _, c = self._borrow()
        return np.ctypeslib.as_array(c, shape=(K,)).copy() if K else np.zeros((0,), np.uint64)


def tq_build_dictionary(mats, top_k: int = 2 ** 16 - 1) -> Dict:
    arrs = [np.ascontiguousarray(m).view(np.uint8).reshape(-1) for m in mats]
    n = len(arrs)
    ptrs = (C.POINTER(C.c_uint8) * max(n, 1))(*[_np_ptr(a, C.c_uint8) for a in arrs])
    lens = (C.c_uint64 * max(n, 1))(*[a.size for a in arrs])
    out = C.c_void_p()
    _check(_lib.tq_build_dictionary(ptrs, lens, n, top_k, C.byref(out)), "tq_build_dictionary")
    return Dict(out.value)


def tq_build_dictionary_device(mats, top_k: int = 2 ** 16 - 1, stream=None) -> Dict:
    """mats: CUDA 1-byte tensors (levels).  Counts the windows on the GPU; same table as tq_build_dictionary."""
    n = len(mats)
    assert n >= 1
    for m in mats:
        assert m.is_cuda and m.is_contiguous() and m.element_size() == 1
    lens = (C.c_uint64 * n)(*[m.numel() for m in mats])
    need = C.c_uint64()
    _check(_lib.tq_build_dictionary_device_size(lens, n, C.byref(need)), "tq_build_dictionary_device_size")
    ws = torch.empty(need.value, dtype=torch.uint8, device=mats[0].device)
    ptrs = (C.c_void_p * n)(*[m.data_ptr() for m in mats])
    out = C.c_void_p()
    with torch.cuda.device(ws.device):
        _check(_lib.tq_build_dictionary_device(ptrs, lens, n, top_k, ws.data_ptr(), ws.numel(), _stream_ptr(stream),
                                               C.byref(out)), "tq_build_dictionary_device")
    return Dict(out.value)


def tq_dict_from_entries(entries: np.ndarray) -> Dict:
    e = np.ascontiguousarray(entries, dtype=np.uint8).reshape(-1, 4)
    out = C.c_void_p()
    _check(_lib.tq_dict_from_entries(_np_ptr(e, C.c_uint8), e.shape[0], C.byref(out)), "tq_dict_from_entries")
    return Dict(out.value)


def tq_encode(d: Dict, codes: np.ndarray):
    """-> (stream uint16, n_hits, n_miss)"""
    w = np.ascontiguousarray(codes).view(np.uint8).reshape(-1)
    n, h, m = C.c_uint64(), C.c_uint64(), C.c_uint64()
    _check(_lib.tq_encode(d._h, _np_ptr(w, C.c_uint8), w.size, None, 0, C.byref(n), C.byref(h), C.byref(m)), "tq_encode")
    out = np.empty(n.value, dtype=np.uint16)
    _check(_lib.tq_encode(d._h, _np_ptr(w, C.c_uint8), w.size, _np_ptr(out, C.c_uint16), out.size,
                          C.byref(n), C.byref(h), C.byref(m)), "tq_encode")
    return out, h.value, m.value


# ------------------------------------------------------------------------------ device
class DeviceDict:
    """A table resident on the GPU: owns the torch buffer and the tq_ddict handle."""

    def __init__(self, handle: int, buf: torch.Tensor, K: int):
        self._h = C.c_void_p(handle)
        self.buf = buf
        self.K = K

    def __del__(self):
        if getattr(self, "_h", None) and _lib is not None:
            _lib.tq_ddict_free(self._h)
            self._h = None


def tq_dict_upload(d: Dict, device="cuda", stream=None) -> DeviceDict:
    need = C.c_uint64()
    _check(_lib.tq_dict_upload_size(d._h, C.byref(need)), "tq_dict_upload_size")
    buf = torch.empty(need.value, dtype=torch.uint8, device=device)
    out = C.c_void_p()
    with torch.cuda.device(buf.device):
        _check(_lib.tq_dict_upload(d._h, buf.data_ptr(), buf.numel(), _stream_ptr(stream), C.byref(out)), "tq_dict_upload")
    return DeviceDict(out.value, buf, d.K)


@dataclass
class MatInfo:
    rows: int
    cols: int
    K: int
    layout: int
    levels_signed: int
    n_hits: int
    n_miss: int
    stream_bytes: int
    payload_bytes: int
    device_bytes: int
    n_raw_words: int


class DeviceMatrix:
    """One compressed matrix resident on the GPU: owns the torch buffer and the tq_dmat handle."""

    def __init__(self, handle: int, buf: torch.Tensor, ddict: DeviceDict):
        self._h = C.c_void_p(handle)
        self.buf = buf
        self.ddict = ddict  # keeps the table alive
        i = _Info()
        _check(_lib.tq_dmat_get_info(self._h, C.byref(i)), "tq_dmat_get_info")
        self.info = MatInfo(*(getattr(i, f[0]) for f in _Info._fields_))

    def __del__(self):
        if getattr(self, "_h", None) and _lib is not None:
            _lib.tq_dmat_free(self._h)
            self._h = None


def tq_upload_size(stream: np.ndarray, rows: int, cols: int, layout: int = TQ_LAYOUT_STREAM) -> int:
    s = np.ascontiguousarray(stream, dtype=np.uint16)
    need = C.c_uint64()
    _check(_lib.tq_upload_size(_np_ptr(s, C.c_uint16), s.size, rows, cols, layout, C.byref(need)), "tq_upload_size")
    return need.value


def tq_upload(ddict: DeviceDict, stream: np.ndarray, rows: int, cols: int, row_scale: np.ndarray,
              row_zero=None, levels_signed: bool = True, layout: int = TQ_LAYOUT_STREAM,
              cuda_stream=None) -> DeviceMatrix:
    s = np.ascontiguousarray(stream, dtype=np.uint16)
    sc = np.ascontiguousarray(row_scale, dtype=np.float32)
    assert sc.size == rows
    zp = None
    if row_zero is not None:
        zr = np.ascontiguousarray(row_zero, dtype=np.float32)
        assert zr.size == rows
        zp = _np_ptr(zr, C.c_float)
    need = C.c_uint64()
    _check(_lib.tq_upload_size(_np_ptr(s, C.c_uint16), s.size, rows, cols, layout, C.byref(need)), "tq_upload_size")
    buf = torch.empty(need.value, dtype=torch.uint8, device=ddict.buf.device)
    out = C.c_void_p()
    with torch.cuda.device(buf.device):
        _check(_lib.tq_upload(ddict._h, _np_ptr(s, C.c_uint16), s.size, rows, cols, _np_ptr(sc, C.c_float), zp,
                              int(levels_signed), layout, buf.data_ptr(), buf.numel(), _stream_ptr(cuda_stream),
                              C.byref(out)), "tq_upload")
    return DeviceMatrix(out.value, buf, ddict)


def tq_upload_device(ddict: DeviceDict, levels: torch.Tensor, row_scale: torch.Tensor, row_zero: torch.Tensor | None = None,
                     levels_signed: bool = True, cuda_stream=None) -> DeviceMatrix:
    """levels: CUDA int8/uint8 [rows][cols]; row_scale / row_zero: CUDA fp32 [rows].  Builds the TILES
    image on the GPU, in a buffer sized for the worst case (info.device_bytes tells what is in use)."""
    assert levels.is_cuda and levels.is_contiguous() and levels.element_size() == 1 and levels.dim() == 2
    assert row_scale.is_cuda and row_scale.dtype == torch.float32 and row_scale.is_contiguous()
    rows, cols = levels.shape
    assert row_scale.numel() == rows
    if row_zero is not None:
        assert row_zero.is_cuda and row_zero.dtype == torch.float32 and row_zero.is_contiguous() and row_zero.numel() == rows
    need = C.c_uint64()
    _check(_lib.tq_upload_device_size(rows, cols, C.byref(need)), "tq_upload_device_size")
    buf = torch.empty(need.value, dtype=torch.uint8, device=levels.device)
    out = C.c_void_p()
    with torch.cuda.device(buf.device):
        _check(_lib.tq_upload_device(ddict._h, levels.data_ptr(), rows, cols, row_scale.data_ptr(),
                                     row_zero.data_ptr() if row_zero is not None else None, int(levels_signed),
                                     buf.data_ptr(), buf.numel(), _stream_ptr(cuda_stream), C.byref(out)), "tq_upload_device")
    return DeviceMatrix(out.value, buf, ddict)


def tq_upload_device_rows(ddict: DeviceDict, levels: torch.Tensor, row_begin: int, row_end: int, row_scale: torch.Tensor,
                          row_zero: torch.Tensor | None = None, levels_signed: bool = True, cuda_stream=None) -> DeviceMatrix:
    """Rows row_begin .. row_end-1 of `levels` (CUDA int8/uint8 [rows][cols]) as a compressed matrix of their
    own; row_scale / row_zero are the full [rows] arrays."""
    assert levels.is_cuda and levels.is_contiguous() and levels.element_size() == 1 and levels.dim() == 2
    rows, cols = levels.shape
    assert row_scale.is_cuda and row_scale.dtype == torch.float32 and row_scale.is_contiguous() and row_scale.numel() == rows
    if row_zero is not None:
        assert row_zero.is_cuda and row_zero.dtype == torch.float32 and row_zero.is_contiguous() and row_zero.numel() == rows
    need = C.c_uint64()
    _check(_lib.tq_upload_device_size(max(row_end - row_begin, 1), cols, C.byref(need)), "tq_upload_device_size")
    buf = torch.empty(need.value, dtype=torch.uint8, device=levels.device)
    out = C.c_void_p()
    with torch.cuda.device(buf.device):
        _check(_lib.tq_upload_device_rows(ddict._h, levels.data_ptr(), rows, cols, row_begin, row_end, row_scale.data_ptr(),
                                          row_zero.data_ptr() if row_zero is not None else None, int(levels_signed),
                                          buf.data_ptr(), buf.numel(), _stream_ptr(cuda_stream), C.byref(out)), "tq_upload_device_rows")
    return DeviceMatrix(out.value, buf, ddict)


def tq_tiles_image_host(d: Dict, stream: np.ndarray, rows: int, cols: int, row_scale: np.ndarray, row_zero=None):
    """-> (image uint8, dict of byte offsets, tiles per row block, row blocks)"""
    s = np.ascontiguousarray(stream, dtype=np.uint16)
    sc = np.ascontiguousarray(row_scale, dtype=np.float32)
    zp = None
    if row_zero is not None:
        zr = np.ascontiguousarray(row_zero, dtype=np.float32)
        zp = _np_ptr(zr, C.c_float)
    need = C.c_uint64()
    _check(_lib.tq_tiles_image_host(d._h, _np_ptr(s, C.c_uint16), s.size, rows, cols, None, None, None, 0,
                                    C.byref(need), None, None), "tq_tiles_image_host")
    out = np.zeros(need.value, dtype=np.uint8)
    offs = (C.c_uint64 * 5)()
    dims = (C.c_uint32 * 2)()
    _check(_lib.tq_tiles_image_host(d._h, _np_ptr(s, C.c_uint16), s.size, rows, cols, _np_ptr(sc, C.c_float), zp,
                                    _np_ptr(out, C.c_uint8), out.size, C.byref(need), offs, dims), "tq_tiles_image_host")
    names = ("scale", "zero", "tile_raw", "tokens", "raw")
    return out, dict(zip(names, (int(o) for o in offs))), int(dims[0]), int(dims[1])


def tq_decompress(m: DeviceMatrix, out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    if out is None:
        out = torch.empty((m.info.rows, m.info.cols), dtype=torch.uint8, device=m.buf.device)
    assert out.is_cuda and out.is_contiguous() and out.numel() == m.info.rows * m.info.cols and out.element_size() == 1
    _check(_lib.tq_decompress(m._h, out.data_ptr(), _stream_ptr(stream)), "tq_decompress")
    return out


def tq_fused_gemv(m: DeviceMatrix, x: torch.Tensor, y: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous()
    x2 = x.view(-1, m.info.cols)
    B = x2.shape[0]
    if y is None:
        y = torch.empty((B, m.info.rows), dtype=torch.float32, device=x.device)
    assert y.is_cuda and y.dtype == torch.float32 and y.is_contiguous() and y.numel() == B * m.info.rows
    _check(_lib.tq_fused_gemv(m._h, x2.data_ptr(), B, y.data_ptr(), _stream_ptr(stream)), "tq_fused_gemv")
    return y


def tq_fused_gemv_host(m: DeviceMatrix, h_x: torch.Tensor, h_y: torch.Tensor, d_x_stage: torch.Tensor,
                       d_y_stage: torch.Tensor, stream=None) -> None:
    """h_x: CPU (pinned) bf16 [B][cols]; h_y: CPU (pinned) fp32 [B][rows]; stages: CUDA tensors."""
    assert (not h_x.is_cuda) and h_x.dtype == torch.bfloat16 and h_x.is_contiguous()
    assert (not h_y.is_cuda) and h_y.dtype == torch.float32 and h_y.is_contiguous()
    B = h_x.numel() // m.info.cols
    assert d_x_stage.is_cuda and d_x_stage.numel() * d_x_stage.element_size() >= B * m.info.cols * 2
    assert d_y_stage.is_cuda and d_y_stage.numel() * d_y_stage.element_size() >= B * m.info.rows * 4
    _check(_lib.tq_fused_gemv_host(m._h, h_x.data_ptr(), B, h_y.data_ptr(), d_x_stage.data_ptr(),
                                   d_y_stage.data_ptr(), _stream_ptr(stream)), "tq_fused_gemv_host")


def tq_fused_gemv_host_static(m: DeviceMatrix, h_x: torch.Tensor, h_y: torch.Tensor, stream=None) -> None:
    """tq_fused_gemv_host without caller staging: the library's built-in 1.5 MiB staging array is
    used, nothing is allocated (B * cols and B * rows are limited to 262144 each)."""
    assert (not h_x.is_cuda) and h_x.dtype == torch.bfloat16 and h_x.is_contiguous()
    assert (not h_y.is_cuda) and h_y.dtype == torch.float32 and h_y.is_contiguous()
    B = h_x.numel() // m.info.cols
    assert h_y.numel() == B * m.info.rows
    with torch.cuda.device(m.buf.device):
        rc = _lib.tq_fused_gemv_host_static(m._h, h_x.data_ptr(), B, h_y.data_ptr(), _stream_ptr(stream))
    if rc == TQ_ERR_UNSUPPORTED_SHAPE:  # the library left the limits in its error text
        raise TqError(rc, "tq_fused_gemv_host_static", _lib.tq_last_cuda_error().decode())
    _check(rc, "tq_fused_gemv_host_static")


def tq_fused_gemm(m: DeviceMatrix, X: torch.Tensor, Y: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.is_contiguous()
    X2 = X.view(-1, m.info.cols)
    M = X2.shape[0]
    if Y is None:
        Y = torch.empty((M, m.info.rows), dtype=torch.float32, device=X.device)
    assert Y.is_cuda and Y.dtype == torch.float32 and Y.is_contiguous() and Y.numel() == M * m.info.rows
    _check(_lib.tq_fused_gemm(m._h, X2.data_ptr(), M, Y.data_ptr(), _stream_ptr(stream)), "tq_fused_gemm")
    return Y


def tq_gemm_workspace_size(m: DeviceMatrix) -> int:
    need = C.c_uint64()
    _check(_lib.tq_gemm_workspace_size(m._h, C.byref(need)), "tq_gemm_workspace_size")
    return need.value


def tq_fused_gemm_ws(m: DeviceMatrix, X: torch.Tensor, workspace: torch.Tensor, Y: torch.Tensor | None = None,
                     stream=None) -> torch.Tensor:
    """Two-phase prefill product for the TILES layout; workspace: CUDA tensor of >= tq_gemm_workspace_size(m) bytes."""
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.is_contiguous() and workspace.is_cuda
    X2 = X.view(-1, m.info.cols)
    M = X2.shape[0]
    if Y is None:
        Y = torch.empty((M, m.info.rows), dtype=torch.float32, device=X.device)
    assert Y.is_cuda and Y.dtype == torch.float32 and Y.is_contiguous() and Y.numel() == M * m.info.rows
    _check(_lib.tq_fused_gemm_ws(m._h, X2.data_ptr(), M, Y.data_ptr(), workspace.data_ptr(),
                                 workspace.numel() * workspace.element_size(), _stream_ptr(stream)), "tq_fused_gemm_ws")
    return Y


def tq_decode_bf16(m: DeviceMatrix, workspace: torch.Tensor, stream=None) -> None:
    assert workspace.is_cuda
    _check(_lib.tq_decode_bf16(m._h, workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                               _stream_ptr(stream)), "tq_decode_bf16")


def tq_gemm_bf16_ws(m: DeviceMatrix, X: torch.Tensor, workspace: torch.Tensor, Y: torch.Tensor | None = None,
                    stream=None) -> torch.Tensor:
    """Phase 2 alone: workspace was filled for m by tq_decode_bf16 or tq_decode_bf16_stack."""
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.is_contiguous() and workspace.is_cuda
    assert workspace.numel() * workspace.element_size() >= tq_gemm_workspace_size(m)
    X2 = X.view(-1, m.info.cols)
    M = X2.shape[0]
    if Y is None:
        Y = torch.empty((M, m.info.rows), dtype=torch.float32, device=X.device)
    assert Y.is_cuda and Y.dtype == torch.float32 and Y.is_contiguous() and Y.numel() == M * m.info.rows
    _check(_lib.tq_gemm_bf16_ws(m._h, X2.data_ptr(), M, Y.data_ptr(), workspace.data_ptr(), _stream_ptr(stream)),
           "tq_gemm_bf16_ws")
    return Y


def tq_stack_plan_host(steps, row_blocks, rb_raw, n_ctas: int):
    """-> (segments [(matrix, first row block, end row block)], cta_seg): the work split of a stack, computed on the host."""
    n = len(steps)
    st = np.ascontiguousarray(steps, dtype=np.uint32)
    rbk = np.ascontiguousarray(row_blocks, dtype=np.uint32)
    raws = [np.ascontiguousarray(r, dtype=np.uint32) for r in rb_raw]
    ptrs = (C.POINTER(C.c_uint32) * n)(*[_np_ptr(r, C.c_uint32) for r in raws])
    cap = n + n_ctas
    segs = np.zeros(3 * cap, dtype=np.uint32)
    cta = np.zeros(n_ctas + 1, dtype=np.uint32)
    ns = C.c_uint32()
    _check(_lib.tq_stack_plan_host(n, _np_ptr(st, C.c_uint32), _np_ptr(rbk, C.c_uint32), ptrs, n_ctas,
                                   _np_ptr(segs, C.c_uint32), cap, C.byref(ns), _np_ptr(cta, C.c_uint32)), "tq_stack_plan_host")
    return [tuple(int(v) for v in segs[3 * i: 3 * i + 3]) for i in range(ns.value)], cta.tolist()


class Stack:
    """Several TILES matrices bound to their operands for one persistent launch.  Keeps the
    matrices, the operand tensors and its own device buffer alive."""

    def __init__(self, handle: int, buf: torch.Tensor, mats, xs, ys, B: int):
        self._h = C.c_void_p(handle)
        self.buf, self.mats, self.xs, self.ys, self.B = buf, list(mats), list(xs), list(ys), B

    @property
    def launches(self) -> int:
        return _lib.tq_stack_launches(self._h)

    def __del__(self):
        if getattr(self, "_h", None) and _lib is not None:
            _lib.tq_stack_free(self._h)
            self._h = None


def tq_test_withhold_table_chunk(on: bool) -> None:
    """Test hook: see tq.h."""
    _lib.tq_test_withhold_table_chunk(int(bool(on)))


def tq_stack_create(mats, xs=None, ys=None, stream=None) -> Stack:
    """mats: DeviceMatrix list (TILES layout, one table); xs[i]: CUDA bf16 [B][cols_i]; ys[i]: CUDA fp32 [B][rows_i].
    Without xs / ys the stack serves tq_decompress_stack only."""
    n = len(mats)
    assert n >= 1 and (xs is None) == (ys is None)
    hm = (C.c_void_p * n)(*[m._h for m in mats])
    B, hx, hy = 0, None, None
    if xs is not None:
        assert len(xs) == n and len(ys) == n
        B = xs[0].numel() // mats[0].info.cols
    need = C.c_uint64()
    _check(_lib.tq_stack_size(hm, n, B, C.byref(need)), "tq_stack_size")
    buf = torch.empty(need.value, dtype=torch.uint8, device=mats[0].buf.device)
    if xs is not None:
        for m, x, y in zip(mats, xs, ys):
            assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous() and x.numel() == B * m.info.cols
            assert y.is_cuda and y.dtype == torch.float32 and y.is_contiguous() and y.numel() == B * m.info.rows
        hx = (C.c_void_p * n)(*[x.data_ptr() for x in xs])
        hy = (C.c_void_p * n)(*[y.data_ptr() for y in ys])
    out = C.c_void_p()
    with torch.cuda.device(buf.device):
        _check(_lib.tq_stack_create(hm, hx, hy, n, B, buf.data_ptr(), buf.numel(), _stream_ptr(stream), C.byref(out)),
               "tq_stack_create")
    return Stack(out.value, buf, mats, xs or [], ys or [], B)


def tq_decompress_stack(s: Stack, outs, stream=None) -> None:
    """outs[i]: CUDA 1-byte tensor with rows_i * cols_i elements."""
    assert len(outs) == len(s.mats)
    for m, o in zip(s.mats, outs):
        assert o.is_cuda and o.is_contiguous() and o.element_size() == 1 and o.numel() == m.info.rows * m.info.cols
    ptrs = torch.tensor([o.data_ptr() for o in outs], dtype=torch.int64).to(s.buf.device)
    _check(_lib.tq_decompress_stack(s._h, ptrs.data_ptr(), _stream_ptr(stream)), "tq_decompress_stack")
    s._out_ptrs = ptrs  # keep the pointer array alive until the stream has used it


def tq_decode_bf16_stack(s: Stack, workspaces, stream=None) -> None:
    """workspaces[i]: CUDA tensor of >= tq_gemm_workspace_size(mats[i]) bytes, 256-byte aligned."""
    assert len(workspaces) == len(s.mats)
    for m, w in zip(s.mats, workspaces):
        assert w.is_cuda and w.numel() * w.element_size() >= tq_gemm_workspace_size(m) and w.data_ptr() % 256 == 0
    ptrs = torch.tensor([w.data_ptr() for w in workspaces], dtype=torch.int64).to(s.buf.device)
    _check(_lib.tq_decode_bf16_stack(s._h, ptrs.data_ptr(), _stream_ptr(stream)), "tq_decode_bf16_stack")
    s._ws_ptrs = ptrs  # keep the pointer array alive until the stream has used it


class GemmPlan:
    """Several workspace GEMMs of one token count bound for one persistent launch.  Keeps the
    matrices, operands, workspaces and its own device buffer alive."""

    def __init__(self, handle: int, buf: torch.Tensor, mats, Xs, Ys, workspaces, M: int):
        self._h = C.c_void_p(handle)
        self.buf, self.mats, self.Xs, self.Ys, self.workspaces, self.M = buf, list(mats), list(Xs), list(Ys), list(workspaces), M

    def __del__(self):
        if getattr(self, "_h", None) and _lib is not None:
            _lib.tq_gemm_plan_free(self._h)
            self._h = None


def tq_gemm_plan_create(mats, Xs, workspaces, Ys=None, stream=None) -> GemmPlan:
    """Xs[i]: CUDA bf16 [M][cols_i]; workspaces[i]: filled (now or later, before the run) by tq_decode_bf16(_stack);
    Ys[i]: CUDA fp32 [M][rows_i] (made here when None)."""
    n = len(mats)
    assert n >= 1 and len(Xs) == n and len(workspaces) == n
    M = Xs[0].view(-1, mats[0].info.cols).shape[0]
    dev = Xs[0].device
    if Ys is None:
        Ys = [torch.empty((M, m.info.rows), dtype=torch.float32, device=dev) for m in mats]
    for m, X, Y, w in zip(mats, Xs, Ys, workspaces):
        assert X.is_cuda and X.dtype == torch.bfloat16 and X.is_contiguous() and X.numel() == M * m.info.cols
        assert Y.is_cuda and Y.dtype == torch.float32 and Y.is_contiguous() and Y.numel() == M * m.info.rows
        assert w.is_cuda and w.numel() * w.element_size() >= tq_gemm_workspace_size(m)
    need = C.c_uint64()
    _check(_lib.tq_gemm_plan_size(n, C.byref(need)), "tq_gemm_plan_size")
    buf = torch.empty(need.value + 256, dtype=torch.uint8, device=dev)
    off = (-buf.data_ptr()) % 256
    arr = lambda ts: (C.c_void_p * n)(*[t.data_ptr() for t in ts])  # noqa: E731
    out = C.c_void_p()
    with torch.cuda.device(dev):
        _check(_lib.tq_gemm_plan_create((C.c_void_p * n)(*[m._h for m in mats]), arr(Xs), arr(Ys), arr(workspaces), n, M,
                                        buf.data_ptr() + off, need.value, _stream_ptr(stream), C.byref(out)),
               "tq_gemm_plan_create")
    return GemmPlan(out.value, buf, mats, Xs, Ys, workspaces, M)


def tq_gemm_plan_run(p: GemmPlan, stream=None) -> None:
    _check(_lib.tq_gemm_plan_run(p._h, _stream_ptr(stream)), "tq_gemm_plan_run")


def tq_gemm_plan_status(p: GemmPlan, stream=None) -> int:
    st = C.c_uint32()
    _check(_lib.tq_gemm_plan_status(p._h, _stream_ptr(stream), C.byref(st)), "tq_gemm_plan_status")
    return st.value


def tq_fused_gemv_stack(s: Stack, stream=None) -> None:
    _check(_lib.tq_fused_gemv_stack(s._h, _stream_ptr(stream)), "tq_fused_gemv_stack")


def tq_fused_gemv_stack_host(s: Stack, h_x: torch.Tensor, d_x_arena: torch.Tensor, h_y: torch.Tensor,
                             d_y_arena: torch.Tensor, stream=None) -> None:
    """h_x / h_y: CPU (pinned) images of the x / y arenas the stack's operands live in."""
    assert (not h_x.is_cuda) and (not h_y.is_cuda) and d_x_arena.is_cuda and d_y_arena.is_cuda
    xb = d_x_arena.numel() * d_x_arena.element_size()
    yb = d_y_arena.numel() * d_y_arena.element_size()
    assert h_x.numel() * h_x.element_size() == xb and h_y.numel() * h_y.element_size() == yb
    _check(_lib.tq_fused_gemv_stack_host(s._h, h_x.data_ptr(), d_x_arena.data_ptr(), xb, h_y.data_ptr(),
                                         d_y_arena.data_ptr(), yb, _stream_ptr(stream)), "tq_fused_gemv_stack_host")


def tq_device_status(m: DeviceMatrix, stream=None) -> int:
    st = C.c_uint32()
    _check(_lib.tq_device_status(m._h, _stream_ptr(stream), C.byref(st)), "tq_device_status")
    return st.value
