"""CPU oracle for the low-bit tensor-parallel synchronisation codec.

TEST INFRASTRUCTURE.  Only the tests, the smoke check and the benchmark's CPU
baseline may import this package; the CUDA library never does.  ``c`` wraps the
scalar C statement (``tpq_oracle.c``, compiled here with gcc), ``oracle_np`` is
the NumPy statement.  Neither shares code with the CUDA path.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

from . import oracle_np  # noqa: F401

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "tpq_oracle.c"
_LIB = _HERE / "libtpq_oracle.so"


def build(force: bool = False) -> Path:
    """Compile the C oracle (gcc, no contraction, no fast-math)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-fPIC", "-shared", "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _ptr(a: np.ndarray, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


class COracle:
    """Thin ctypes front end of tpq_oracle.c (argument marshalling only)."""

    def __init__(self):
        self.lib = ctypes.CDLL(str(build()))
        L = self.lib
        i64, f32 = ctypes.c_int64, ctypes.c_float
        u16p, f32p = ctypes.POINTER(ctypes.c_uint16), ctypes.POINTER(ctypes.c_float)
        i32p, u8p = ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_uint8)
        L.tpqo_num_threads.restype = ctypes.c_int
        L.tpqo_colminmax.argtypes = [u16p, i64, i64, i64, f32p, f32p]
        L.tpqo_calibrate.argtypes = [f32p, f32p, ctypes.POINTER(i64), u16p, i64, i64, i64, i64, f32]
        L.tpqo_ranges.argtypes = [f32p, f32p, i64, i64, f32p, f32p]
        L.tpqo_select.argtypes = [f32p, i64, i64, i32p]
        L.tpqo_default_k.argtypes = [i64]
        L.tpqo_default_k.restype = i64
        L.tpqo_params.argtypes = [f32p, i64, f32p, f32p]
        L.tpqo_lp_bytes.argtypes = [i64, i64, i64]
        L.tpqo_lp_bytes.restype = i64
        L.tpqo_payload_bytes.argtypes = [i64, i64, i64]
        L.tpqo_payload_bytes.restype = i64
        L.tpqo_slot_order.argtypes = [i64, i32p, i64, i32p]
        L.tpqo_quantize_one.argtypes = [ctypes.c_uint16, f32]
        L.tpqo_quantize_one.restype = ctypes.c_int
        L.tpqo_quantize_pack.argtypes = [u16p, i64, i64, i64, i32p, i64, f32p, u8p]
        L.tpqo_dequant_reduce.argtypes = [ctypes.POINTER(u8p), i64, i64, i64, i32p, i64, f32p,
                                          ctypes.POINTER(ctypes.c_double), f32p]
        L.tpqo_round_bf16_f32.argtypes = [f32p, i64, u16p]
        ci = ctypes.c_int
        L.tpqo_params_b.argtypes = [f32p, i64, ci, f32p, f32p]
        L.tpqo_lp_bytes_b.argtypes = [i64, i64, i64, ci]
        L.tpqo_lp_bytes_b.restype = i64
        L.tpqo_payload_bytes_b.argtypes = [i64, i64, i64, ci]
        L.tpqo_payload_bytes_b.restype = i64
        L.tpqo_quantize_one_b.argtypes = [ctypes.c_uint16, f32, ci]
        L.tpqo_quantize_one_b.restype = ctypes.c_int
        L.tpqo_quantize_pack_b.argtypes = [u16p, i64, i64, i64, i32p, i64, f32p, ci, u8p]
        L.tpqo_dequant_reduce_b.argtypes = [ctypes.POINTER(u8p), i64, i64, i64, i32p, i64, f32p, ci,
                                            ctypes.POINTER(ctypes.c_double), f32p]
        L.tpqo_dequant_reduce_bias_b.argtypes = [ctypes.POINTER(u8p), i64, i64, i64, i32p, i64, f32p, ci, f32p,
                                                 ctypes.POINTER(ctypes.c_double), f32p]

    def num_threads(self) -> int:
        return int(self.lib.tpqo_num_threads())

    # ---- calibration
    def col_minmax(self, y_bits: np.ndarray):
        y = np.ascontiguousarray(y_bits, dtype=np.uint16)
        S, E = y.shape
        mn = np.empty(E, np.float32)
        mx = np.empty(E, np.float32)
        self.lib.tpqo_colminmax(_ptr(y, ctypes.c_uint16), S, E, E, _ptr(mn, ctypes.c_float),
                                _ptr(mx, ctypes.c_float))
        return mn, mx

    def calibrate(self, m, M, count: int, y_bits: np.ndarray, gamma: float):
        y = np.ascontiguousarray(y_bits, dtype=np.uint16)
        n_seq, S, E = y.shape
        m = np.zeros(E, np.float32) if m is None else np.array(m, dtype=np.float32, copy=True)
        M = np.zeros(E, np.float32) if M is None else np.array(M, dtype=np.float32, copy=True)
        cnt = ctypes.c_int64(count)
        self.lib.tpqo_calibrate(_ptr(m, ctypes.c_float), _ptr(M, ctypes.c_float), ctypes.byref(cnt),
                                _ptr(y, ctypes.c_uint16), n_seq, S, E, E, ctypes.c_float(gamma))
        return m, M, int(cnt.value)

    def ranges(self, m: np.ndarray, M: np.ndarray):
        m = np.ascontiguousarray(m, dtype=np.float32)
        M = np.ascontiguousarray(M, dtype=np.float32)
        N, E = m.shape
        R = np.empty((N, E), np.float32)
        Rbar = np.empty(E, np.float32)
        self.lib.tpqo_ranges(_ptr(m, ctypes.c_float), _ptr(M, ctypes.c_float), N, E,
                             _ptr(R, ctypes.c_float), _ptr(Rbar, ctypes.c_float))
        return R, Rbar

    def default_k(self, E: int) -> int:
        return int(self.lib.tpqo_default_k(E))

    def select(self, Rbar: np.ndarray, k: int) -> np.ndarray:
        Rbar = np.ascontiguousarray(Rbar, dtype=np.float32)
        out = np.empty(max(k, 1), np.int32)
        self.lib.tpqo_select(_ptr(Rbar, ctypes.c_float), Rbar.shape[0], k, _ptr(out, ctypes.c_int32))
        return out[:k].copy()

    def params(self, R: np.ndarray, bits: int = 4):
        R = np.ascontiguousarray(R, dtype=np.float32)
        s = np.empty_like(R)
        inv_s = np.empty_like(R)
        if bits == 4:
            self.lib.tpqo_params(_ptr(R, ctypes.c_float), R.size, _ptr(s, ctypes.c_float),
                                 _ptr(inv_s, ctypes.c_float))
        else:
            self.lib.tpqo_params_b(_ptr(R, ctypes.c_float), R.size, bits, _ptr(s, ctypes.c_float),
                                   _ptr(inv_s, ctypes.c_float))
        return s, inv_s

    # ---- payload
    def lp_bytes(self, T: int, E: int, k: int, bits: int = 4) -> int:
        if bits == 4:
            return int(self.lib.tpqo_lp_bytes(T, E, k))
        return int(self.lib.tpqo_lp_bytes_b(T, E, k, bits))

    def payload_bytes(self, T: int, E: int, k: int, bits: int = 4) -> int:
        if bits == 4:
            return int(self.lib.tpqo_payload_bytes(T, E, k))
        return int(self.lib.tpqo_payload_bytes_b(T, E, k, bits))

    def lp_index(self, E: int, hp_idx) -> np.ndarray:
        """Feature held by each code slot (the payload's slot order)."""
        hp = np.ascontiguousarray(hp_idx, dtype=np.int32)
        k = hp.shape[0]
        out = np.empty(max(E - k, 1), np.int32)
        hp_arg = hp if k else np.zeros(1, np.int32)
        self.lib.tpqo_slot_order(E, _ptr(hp_arg, ctypes.c_int32), k, _ptr(out, ctypes.c_int32))
        return out[: E - k].copy()

    def quantize_one(self, x_bits: int, inv_s: float, bits: int = 4) -> int:
        if bits == 4:
            return int(self.lib.tpqo_quantize_one(ctypes.c_uint16(int(x_bits)), ctypes.c_float(inv_s)))
        return int(self.lib.tpqo_quantize_one_b(ctypes.c_uint16(int(x_bits)), ctypes.c_float(inv_s), bits))

    def quantize_pack(self, y_bits: np.ndarray, hp_idx: np.ndarray, inv_s: np.ndarray, bits: int = 4) -> np.ndarray:
        y = np.ascontiguousarray(y_bits, dtype=np.uint16)
        T, E = y.shape
        hp = np.ascontiguousarray(hp_idx, dtype=np.int32)
        k = hp.shape[0]
        inv = np.ascontiguousarray(inv_s, dtype=np.float32)
        assert inv.shape == (E,)
        out = np.empty(self.payload_bytes(T, E, k, bits), np.uint8)
        hp_arg = hp if k else np.zeros(1, np.int32)
        if bits == 4:
            self.lib.tpqo_quantize_pack(_ptr(y, ctypes.c_uint16), T, E, E, _ptr(hp_arg, ctypes.c_int32), k,
                                        _ptr(inv, ctypes.c_float), _ptr(out, ctypes.c_uint8))
        else:
            self.lib.tpqo_quantize_pack_b(_ptr(y, ctypes.c_uint16), T, E, E, _ptr(hp_arg, ctypes.c_int32), k,
                                          _ptr(inv, ctypes.c_float), bits, _ptr(out, ctypes.c_uint8))
        return out

    def dequant_reduce(self, payloads, T: int, E: int, hp_idx: np.ndarray, s: np.ndarray,
                       want_chain32: bool = True, bits: int = 4, bias=None):
        N = len(payloads)
        hp = np.ascontiguousarray(hp_idx, dtype=np.int32)
        k = hp.shape[0]
        s = np.ascontiguousarray(s, dtype=np.float32)
        assert s.shape == (N, E)
        pls = [np.ascontiguousarray(p, dtype=np.uint8) for p in payloads]
        for p in pls:
            assert p.size == self.payload_bytes(T, E, k, bits)
        u8p = ctypes.POINTER(ctypes.c_uint8)
        arr = (u8p * N)(*[_ptr(p, ctypes.c_uint8) for p in pls])
        ref = np.empty((T, E), np.float64)
        chain = np.empty((T, E), np.float32) if want_chain32 else None
        hp_arg = hp if k else np.zeros(1, np.int32)
        if bias is not None:
            b = np.ascontiguousarray(bias, dtype=np.float32)
            assert b.shape == (E,)
            self.lib.tpqo_dequant_reduce_bias_b(arr, N, T, E, _ptr(hp_arg, ctypes.c_int32), k, _ptr(s, ctypes.c_float),
                                                bits, _ptr(b, ctypes.c_float), _ptr(ref, ctypes.c_double),
                                                _ptr(chain, ctypes.c_float) if want_chain32 else None)
        elif bits == 4:
            self.lib.tpqo_dequant_reduce(arr, N, T, E, _ptr(hp_arg, ctypes.c_int32), k, _ptr(s, ctypes.c_float),
                                         _ptr(ref, ctypes.c_double),
                                         _ptr(chain, ctypes.c_float) if want_chain32 else None)
        else:
            self.lib.tpqo_dequant_reduce_b(arr, N, T, E, _ptr(hp_arg, ctypes.c_int32), k, _ptr(s, ctypes.c_float),
                                           bits, _ptr(ref, ctypes.c_double),
                                           _ptr(chain, ctypes.c_float) if want_chain32 else None)
        return ref, chain

    def linear_bf16(self, x_bits: np.ndarray, w_bits: np.ndarray) -> np.ndarray:
        """Section 2: y = bf16(x W^T), x [T][K], w [E][K] BF16 patterns; exact sum, one rounding."""
        x = np.ascontiguousarray(x_bits, dtype=np.uint16)
        w = np.ascontiguousarray(w_bits, dtype=np.uint16)
        T, K = x.shape
        E, K2 = w.shape
        assert K == K2
        y = np.empty((T, E), np.uint16)
        self.lib.tpqo_linear_bf16(_ptr(x, ctypes.c_uint16), _ptr(w, ctypes.c_uint16), T, K, E, _ptr(y, ctypes.c_uint16))
        return y

    def round_bf16(self, x: np.ndarray) -> np.ndarray:
        x = np.ascontiguousarray(x, dtype=np.float32)
        out = np.empty(x.shape, np.uint16)
        self.lib.tpqo_round_bf16_f32(_ptr(x, ctypes.c_float), x.size, _ptr(out, ctypes.c_uint16))
        return out


_c = None


def c() -> COracle:
    """The process-wide C oracle (compiled on first use)."""
    global _c
    if _c is None:
        _c = COracle()
    return _c
