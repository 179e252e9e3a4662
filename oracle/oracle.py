"""ctypes front end of the CPU oracle (tq_oracle.c) -- TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this module.  It shares nothing with the CUDA library: it compiles and loads its
own shared object from tq_oracle.c with gcc.

Every function cites the passage of the paper it follows; the arithmetic lives
in the C file, this module only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "tq_oracle.c"
_LIB = _HERE / "libtq_oracle.so"

ESCAPE = 0xFFFF
MAX_ENTRIES = 65534


def build(force: bool = False) -> Path:
    """Compile tq_oracle.c (plain C, no fast-math, no FMA contraction)."""
    if force or (not _LIB.exists()) or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fno-fast-math",
             "-ffp-contract=off", "-o", str(tmp), str(_SRC), "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _L():
    global _lib
    if _lib is None:
        lib = C.CDLL(str(build()))
        u8p, u16p, u64p = C.POINTER(C.c_uint8), C.POINTER(C.c_uint16), C.POINTER(C.c_uint64)
        f32p, f64p = C.POINTER(C.c_float), C.POINTER(C.c_double)
        lib.tqo_quantize_paper.argtypes = [f32p, C.c_uint64, u8p, f32p, f32p]
        lib.tqo_quantize_paper.restype = C.c_int
        lib.tqo_quantize_paper_bits.argtypes = [f32p, C.c_uint64, C.c_int, u8p, f32p, f32p]
        lib.tqo_quantize_paper_bits.restype = C.c_int
        lib.tqo_quantize_rows.argtypes = [f32p, C.c_uint32, C.c_uint32, C.POINTER(C.c_int8), f32p]
        lib.tqo_quantize_rows.restype = None
        lib.tqo_build_dictionary.argtypes = [C.POINTER(u8p), u64p, C.c_int, C.c_uint32]
        lib.tqo_build_dictionary.restype = C.c_void_p
        lib.tqo_dict_from_entries.argtypes = [u8p, C.c_uint32]
        lib.tqo_dict_from_entries.restype = C.c_void_p
        lib.tqo_build_dictionary_seq.argtypes = [C.POINTER(u8p), u64p, C.c_int, C.c_uint32, C.c_uint32]
        lib.tqo_build_dictionary_seq.restype = C.c_void_p
        lib.tqo_dict_from_entries_seq.argtypes = [u8p, C.c_uint32, C.c_uint32]
        lib.tqo_dict_from_entries_seq.restype = C.c_void_p
        lib.tqo_dict_seq.argtypes = [C.c_void_p]
        lib.tqo_dict_seq.restype = C.c_uint32
        lib.tqo_dict_free.argtypes = [C.c_void_p]
        lib.tqo_dict_free.restype = None
        lib.tqo_dict_size.argtypes = [C.c_void_p]
        lib.tqo_dict_size.restype = C.c_uint32
        lib.tqo_dict_entries.argtypes = [C.c_void_p]
        lib.tqo_dict_entries.restype = u8p
        lib.tqo_dict_counts.argtypes = [C.c_void_p]
        lib.tqo_dict_counts.restype = u64p
        lib.tqo_dict_distinct.argtypes = [C.c_void_p]
        lib.tqo_dict_distinct.restype = C.c_uint64
        lib.tqo_dict_windows.argtypes = [C.c_void_p]
        lib.tqo_dict_windows.restype = C.c_uint64
        lib.tqo_encode.argtypes = [C.c_void_p, u8p, C.c_uint64, u16p, C.c_uint64, u64p, u64p]
        lib.tqo_encode.restype = C.c_uint64
        lib.tqo_decode.argtypes = [C.c_void_p, u16p, C.c_uint64, u8p, C.c_uint64]
        lib.tqo_decode.restype = C.c_int64
        lib.tqo_layer_forward.argtypes = [u8p, C.c_int, C.c_uint32, C.c_uint32, f32p, f32p,
                                          f64p, C.c_uint32, f64p]
        lib.tqo_layer_forward.restype = None
        _lib = lib
    return _lib


def _ptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(C.POINTER(ctype))


def quantize_paper(x: np.ndarray, bits: int = 8):
    """Listing 1: per-tensor min-max levels 0..2^bits-1 (bits = 8 in the paper's pipeline).
    -> (q uint8, scale, zero)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    q = np.empty(x.shape, dtype=np.uint8)
    s, z = C.c_float(), C.c_float()
    rc = _L().tqo_quantize_paper_bits(_ptr(x, C.c_float), x.size, int(bits), _ptr(q, C.c_uint8),
                                      C.byref(s), C.byref(z))
    if rc != 0:
        raise ValueError("degenerate range (max == min) or bits outside 1..8")
    return q, np.float32(s.value), np.float32(z.value)


def quantize_rows(w: np.ndarray):
    """Benchmark configs' quantizer: per-row symmetric absmax int8.  -> (q int8, scale[rows])."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    rows, cols = w.shape
    q = np.empty((rows, cols), dtype=np.int8)
    s = np.empty(rows, dtype=np.float32)
    _L().tqo_quantize_rows(_ptr(w, C.c_float), rows, cols, _ptr(q, C.c_int8), _ptr(s, C.c_float))
    return q, s


class Dictionary:
    """Listing 2's compression table: K <= 65534 entries of `seq` bytes (Listing 2's sequence_length,
    4 unless stated), code = rank + 1."""

    def __init__(self, handle):
        if not handle:
            raise MemoryError("oracle dictionary allocation failed")
        self._h = C.c_void_p(handle)

    @classmethod
    def build(cls, mats, top_k: int = 2 ** 16 - 1, seq: int = 4) -> "Dictionary":
        arrs = [np.ascontiguousarray(m).view(np.uint8).reshape(-1) for m in mats]
        n = len(arrs)
        ptrs = (C.POINTER(C.c_uint8) * n)(*[_ptr(a, C.c_uint8) for a in arrs])
        lens = (C.c_uint64 * n)(*[a.size for a in arrs])
        if not 1 <= seq <= 8:
            raise ValueError("sequence length must be 1..8")
        return cls(_L().tqo_build_dictionary_seq(ptrs, lens, n, top_k, seq))

    @classmethod
    def from_entries(cls, entries: np.ndarray, seq: int = 4) -> "Dictionary":
        e = np.ascontiguousarray(entries, dtype=np.uint8).reshape(-1, seq)
        return cls(_L().tqo_dict_from_entries_seq(_ptr(e, C.c_uint8), e.shape[0], seq))

    def __del__(self):
        if getattr(self, "_h", None) and _lib is not None:
            _lib.tqo_dict_free(self._h)
            self._h = None

    @property
    def K(self) -> int:
        return int(_L().tqo_dict_size(self._h))

    @property
    def seq(self) -> int:
        return int(_L().tqo_dict_seq(self._h))

    @property
    def entries(self) -> np.ndarray:
        K, L = self.K, self.seq
        if K == 0:
            return np.zeros((0, L), dtype=np.uint8)
        return np.ctypeslib.as_array(_L().tqo_dict_entries(self._h), shape=(K, L)).copy()

    @property
    def counts(self) -> np.ndarray:
        K = self.K
        if K == 0:
            return np.zeros((0,), dtype=np.uint64)
        return np.ctypeslib.as_array(_L().tqo_dict_counts(self._h), shape=(K,)).copy()

    @property
    def n_distinct(self) -> int:
        return int(_L().tqo_dict_distinct(self._h))

    @property
    def n_windows(self) -> int:
        return int(_L().tqo_dict_windows(self._h))

    def encode(self, codes: np.ndarray):
        """Listing 3.  -> (stream uint16, hits, misses)."""
        w = np.ascontiguousarray(codes).view(np.uint8).reshape(-1)
        h, m = C.c_uint64(), C.c_uint64()
        n = _L().tqo_encode(self._h, _ptr(w, C.c_uint8), w.size, None, 0, C.byref(h), C.byref(m))
        out = np.empty(int(n), dtype=np.uint16)
        n2 = _L().tqo_encode(self._h, _ptr(w, C.c_uint8), w.size, _ptr(out, C.c_uint16),
                             out.size, C.byref(h), C.byref(m))
        assert n2 == n
        return out, int(h.value), int(m.value)

    def decode(self, stream: np.ndarray, n_out: int | None = None) -> np.ndarray:
        """Listing 4.  Raises KeyError on an unknown code, as the listing does."""
        s = np.ascontiguousarray(stream, dtype=np.uint16)
        cap = self.seq * s.size + self.seq if n_out is None else n_out
        out = np.empty(cap, dtype=np.uint8)
        n = _L().tqo_decode(self._h, _ptr(s, C.c_uint16), s.size, _ptr(out, C.c_uint8), cap)
        if n == -1:
            raise KeyError("unknown code in stream")
        if n == -2:
            raise ValueError("decoded output larger than expected")
        return out[:n].copy()


def layer_forward(q: np.ndarray, scale: np.ndarray, x: np.ndarray, zero=None) -> np.ndarray:
    """y[b][r] = s_r * sum_c (q[r][c] - z_r) x[b][c] in fp64 (Section 2.3, Listing 1 dequant).

    q: int8 (signed levels) or uint8 (unsigned levels) [rows][cols]; x: [B][cols].
    """
    q = np.ascontiguousarray(q)
    assert q.dtype in (np.int8, np.uint8) and q.ndim == 2
    rows, cols = q.shape
    x = np.ascontiguousarray(x, dtype=np.float64).reshape(-1, cols)
    s = np.ascontiguousarray(scale, dtype=np.float32)
    z = None if zero is None else np.ascontiguousarray(zero, dtype=np.float32)
    y = np.empty((x.shape[0], rows), dtype=np.float64)
    _L().tqo_layer_forward(_ptr(q.view(np.uint8), C.c_uint8), int(q.dtype == np.int8), rows, cols,
                           _ptr(s, C.c_float), None if z is None else _ptr(z, C.c_float),
                           _ptr(x, C.c_double), x.shape[0], _ptr(y, C.c_double))
    return y
