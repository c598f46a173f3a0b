"""NumPy statement of the codec -- TEST INFRASTRUCTURE, not product code.

A second, independently written CPU statement of the method of "Towards Low-bit
Communication for Tensor Parallel LLM Inference" (arXiv 2411.07942), used to
cross-check the scalar C oracle bit for bit and as the readable form of the
algorithm.  It shares nothing with the CUDA library and must never be imported
by it.

BF16 tensors are ``np.uint16`` bit patterns.  Every calibration / parameter /
quantiser operation is one ``np.float32`` operation (NumPy never fuses a
multiply with an add); the reduction reference is ``np.float64``.

Paper passages followed:
  Section 3 "Calibration", Eq. (1)-(2)             -> col_minmax, calibrate
  Section 3, R = 2 max(-m, M); R-bar = sum_i R^(i)  -> ranges
  Section 3 "Selecting High Precision Features"    -> select, default_k (Section 4)
  Section 3 symmetric Int4                          -> params, quantize_codes
  Figure 2, Section 4 bit count                     -> pack, payload_bytes
  Figure 2 caption, Section 5                       -> dequant_reduce
"""
from __future__ import annotations

import numpy as np

F32 = np.float32
LEVELS_MINUS_ONE = F32(15.0)          # 2**4 - 1 steps across the range R
S_FLOOR = F32(2.0 ** -23)             # floor for a degenerate (zero) range
Q_MIN, Q_MAX = F32(-8.0), F32(7.0)    # signed Int4 codes


# ------------------------------------------------------------------ BF16 <-> f32
def widen(bits: np.ndarray) -> np.ndarray:
    """BF16 bit patterns -> float32, exactly."""
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(F32)


def round_bf16(x: np.ndarray) -> np.ndarray:
    """float32 -> BF16 bit patterns, round to nearest even."""
    u = np.asarray(x, dtype=F32).view(np.uint32)
    nan = (u & np.uint32(0x7FFFFFFF)) > np.uint32(0x7F800000)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    r = np.where(nan, (u >> np.uint32(16)) | np.uint32(0x40), r)
    return r.astype(np.uint16)


def round_bf16_f64(v: np.ndarray) -> np.ndarray:
    """float64 -> BF16 bit patterns with ONE rounding (nearest, ties to even); finite inputs within BF16's
    normal range (the layer outputs this is used for)."""
    v = np.asarray(v, dtype=np.float64)
    a = np.abs(v)
    _, e = np.frexp(a)                              # a = f 2^e, 0.5 <= f < 1
    q = np.maximum(e - 8, -133)                     # weight of the last of 8 significant bits
    r = np.rint(np.ldexp(a, -q))                    # exact scaling; rint rounds half to even
    out = np.copysign(np.ldexp(r, q), v).astype(F32)  # representable: the conversion is exact
    return (out.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def linear_bf16(x_bits: np.ndarray, w_bits: np.ndarray) -> np.ndarray:
    """Section 2: y = bf16(x W^T) for x [T][K], w [E][K] given as BF16 patterns.  Products of BF16 values
    are exact in float64; the library matmul sums them in float64; one rounding to BF16."""
    x = widen(x_bits).astype(np.float64)
    w = widen(w_bits).astype(np.float64)
    return round_bf16_f64(x @ w.T)


def _order_key(bits: np.ndarray) -> np.ndarray:
    """Monotone integer key of non-NaN BF16 patterns with -0 below +0."""
    b = np.asarray(bits, dtype=np.uint16).astype(np.int32)
    mag = b & 0x7FFF
    return np.where(b & 0x8000, -mag - 1, mag)


# ------------------------------------------------------------------ calibration
def col_minmax(y_bits: np.ndarray):
    """Eq. (1)-(2): min and max of every feature column over one sequence [S, E]."""
    key = _order_key(y_bits)
    lo = np.take_along_axis(y_bits, key.argmin(axis=0)[None, :], axis=0)[0]
    hi = np.take_along_axis(y_bits, key.argmax(axis=0)[None, :], axis=0)[0]
    return widen(lo), widen(hi)


def calibrate(m, M, count: int, y_bits: np.ndarray, gamma):
    """Fold sequences [n_seq, S, E] of one device into its (m, M), Eq. (1)-(2).

    The first sequence a device sees initialises (m, M); afterwards
    m <- (1-gamma) m + gamma min, literally left to right in float32."""
    gamma = F32(gamma)
    c = F32(F32(1.0) - gamma)
    for seq in y_bits:
        mn, mx = col_minmax(seq)
        if count == 0:
            m, M = mn.copy(), mx.copy()
        else:
            m = (c * m).astype(F32) + (gamma * mn).astype(F32)
            M = (c * M).astype(F32) + (gamma * mx).astype(F32)
        count += 1
    return m.astype(F32), M.astype(F32), count


def ranges(m: np.ndarray, M: np.ndarray):
    """R^(i)_j = 2 max(-m, M) and R-bar_j = sum over devices (ascending, float32)."""
    m = np.asarray(m, dtype=F32)
    M = np.asarray(M, dtype=F32)
    R = (F32(2.0) * np.maximum(-m, M)).astype(F32)
    Rbar = R[0].copy()
    for i in range(1, R.shape[0]):
        Rbar = (Rbar + R[i]).astype(F32)
    return R, Rbar


def default_k(E: int) -> int:
    """Section 4: k = floor(E / 64)."""
    return E // 64


def select(Rbar: np.ndarray, k: int) -> np.ndarray:
    """Top-k features by R-bar; ties to the lower index; returned ascending."""
    E = Rbar.shape[0]
    order = sorted(range(E), key=lambda j: (-float(Rbar[j]), j))
    return np.array(sorted(order[:k]), dtype=np.int32)


def params(R: np.ndarray, bits: int = 4):
    """Step s = R/(2^bits - 1) (R/15 for Int4) floored at 2^-23, and the reciprocal the quantiser uses."""
    levels = LEVELS_MINUS_ONE if bits == 4 else F32((1 << bits) - 1)
    s = (np.asarray(R, dtype=F32) / levels).astype(F32)
    s = np.where(s >= S_FLOOR, s, S_FLOOR).astype(F32)
    inv_s = (F32(1.0) / s).astype(F32)
    return s, inv_s


# ------------------------------------------------------------------ compression
def lp_index(E: int, hp_idx: np.ndarray) -> np.ndarray:
    """Feature held by each of the L = E-k code slots of a token ("hole filling"):
    slot c holds feature c unless c is selected; the selected features below L are
    filled, in ascending order, with the unselected features at or above L."""
    hp = np.asarray(hp_idx, dtype=np.int64)
    L = E - len(hp)
    sel = np.zeros(E, dtype=bool)
    sel[hp] = True
    order = np.arange(L, dtype=np.int32)
    holes = np.nonzero(sel[:L])[0]
    fillers = L + np.nonzero(~sel[L:])[0]
    assert len(holes) == len(fillers)
    order[holes] = fillers
    return order


def quantize_codes(y_bits: np.ndarray, inv_s: np.ndarray, bits: int = 4) -> np.ndarray:
    """Symmetric codes in [-2^(bits-1), 2^(bits-1) - 1] ([-8, 7] for Int4): product rounded to
    float32, clamped, then rounded half-to-even (np.rint)."""
    q_min = Q_MIN if bits == 4 else F32(-(1 << (bits - 1)))
    q_max = Q_MAX if bits == 4 else F32((1 << (bits - 1)) - 1)
    with np.errstate(over="ignore"):
        u = (widen(y_bits) * np.asarray(inv_s, dtype=F32)).astype(F32)
    u = np.minimum(np.maximum(u, q_min), q_max)
    return np.rint(u).astype(np.int16)


def lp_bytes(T: int, E: int, k: int, bits: int = 4) -> int:
    nbits = T * (E - k) * bits
    return ((nbits + 7) // 8 + 15) // 16 * 16


def payload_bytes(T: int, E: int, k: int, bits: int = 4) -> int:
    return lp_bytes(T, E, k, bits) + 2 * T * k


def bits_per_value(T: int, E: int, k: int, bits: int = 4) -> float:
    return 8.0 * payload_bytes(T, E, k, bits) / (T * E)


def quantize_pack(y_bits: np.ndarray, hp_idx: np.ndarray, inv_s: np.ndarray, bits: int = 4) -> np.ndarray:
    """One device's [T, E] BF16 partial sums -> payload bytes.  The codes form one little-endian bit
    stream: bit b of code p is bit p*bits + b of the stream (for Int4: low nibble first)."""
    T, E = y_bits.shape
    k = len(hp_idx)
    lp = lp_index(E, hp_idx)
    codes = quantize_codes(y_bits[:, lp], inv_s[lp], bits).reshape(-1)          # [T (E-k)]
    u = (codes.astype(np.int32) & ((1 << bits) - 1)).astype(np.uint32)
    bitplanes = ((u[:, None] >> np.arange(bits, dtype=np.uint32)[None, :]) & 1).astype(np.uint8)   # [n, bits]
    packed = np.packbits(bitplanes.reshape(-1), bitorder="little")
    out = np.zeros(payload_bytes(T, E, k, bits), dtype=np.uint8)
    out[: packed.size] = packed
    hp = np.ascontiguousarray(y_bits[:, np.asarray(hp_idx, dtype=np.int64)])
    out[lp_bytes(T, E, k, bits):] = hp.view(np.uint8).reshape(-1)
    return out


def unpack(payload: np.ndarray, T: int, E: int, k: int, bits: int = 4):
    """Payload -> (codes [T, E-k] int16, hp [T, k] BF16 bits)."""
    L = E - k
    nb = lp_bytes(T, E, k, bits)
    stream = np.unpackbits(np.asarray(payload[:nb], dtype=np.uint8), bitorder="little")[: T * L * bits]
    planes = stream.reshape(T * L, bits).astype(np.int32)
    u = (planes << np.arange(bits, dtype=np.int32)[None, :]).sum(axis=1)
    codes = np.where(u >= (1 << (bits - 1)), u - (1 << bits), u).astype(np.int16).reshape(T, L)
    hp = payload[nb:].view(np.uint16).reshape(T, k) if k else np.zeros((T, 0), np.uint16)
    return codes, hp


# ------------------------------------------------------------------ decompression + sum
def dequant_reduce(payloads, T: int, E: int, hp_idx: np.ndarray, s: np.ndarray, bits: int = 4, bias=None):
    """Sum over devices of the dequantised payloads, in float64, original feature order."""
    k = len(hp_idx)
    lp = lp_index(E, hp_idx)
    out = np.zeros((T, E), dtype=np.float64)
    for i, p in enumerate(payloads):
        codes, hp = unpack(np.asarray(p, dtype=np.uint8), T, E, k, bits)
        out[:, lp] += codes.astype(np.float64) * s[i, lp].astype(np.float64)[None, :]
        if k:
            out[:, np.asarray(hp_idx, dtype=np.int64)] += widen(hp).astype(np.float64)
    if bias is not None:    # f(x) = sum_i f_i(x_i) + b
        out += np.asarray(bias, dtype=F32).astype(np.float64)[None, :]
    return out
