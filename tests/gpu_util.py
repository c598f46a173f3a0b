"""Helpers of the GPU parity tests: upload seeded inputs, drive the CUDA library
through its C ABI (via the ctypes binding), and compare with the CPU oracle."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from oracle import oracle_np
from paper_2411_07942_b200 import binding, build

CANARY = 0xA5


def ensure_lib():
    build.build()
    return binding.lib()


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    """uint16 BF16 patterns -> device tensor (int16 storage; only the pointer is used)."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda()


def guarded(nbytes: int, pad: int = 4096):
    """A device byte buffer with canary bands before and after; returns (whole, view)."""
    whole = torch.full((nbytes + 2 * pad,), CANARY, dtype=torch.uint8, device="cuda")
    return whole, whole[pad: pad + nbytes]


def guards_intact(whole: torch.Tensor, nbytes: int, pad: int = 4096) -> bool:
    h = whole.cpu().numpy()
    return bool((h[:pad] == CANARY).all() and (h[pad + nbytes:] == CANARY).all())


def calibrate_both(t: binding.Tpq, cal_list, gamma=0.01, chunks=None):
    """cal_list[i] = [n_seq, S, E] uint16.  Returns the oracle's (m, M) after folding the same data."""
    orc = oracle.c()
    ms, Ms = [], []
    for i, cal in enumerate(cal_list):
        n_seq, S, E = cal.shape
        d = dev_bf16(cal)
        if chunks:
            q = 0
            for c in chunks:
                t.calibrate_ranges(i, d.data_ptr() + q * S * E * 2, c, S)
                q += c
            assert q == n_seq
        else:
            t.calibrate_ranges(i, d.data_ptr(), n_seq, S)
        torch.cuda.synchronize()
        m, M, _ = orc.calibrate(None, None, 0, cal, gamma)
        ms.append(m)
        Ms.append(M)
    return np.stack(ms), np.stack(Ms)


def bits_equal(a: np.ndarray, b: np.ndarray) -> bool:
    a = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    b = np.ascontiguousarray(b, dtype=np.float32).view(np.uint32)
    return a.shape == b.shape and bool(np.array_equal(a, b))


def term_abs_sum(payloads, T, E, hp, s, bits=4):
    """sum_i |term_i| per output element (for the cancellation clause of the tolerance)."""
    k = len(hp)
    lp = oracle_np.lp_index(E, hp)
    out = np.zeros((T, E))
    for i, p in enumerate(payloads):
        codes, hpv = oracle_np.unpack(np.asarray(p), T, E, k, bits)
        out[:, lp] += np.abs(codes.astype(np.float64)) * s[i, lp].astype(np.float64)[None, :]
        if k:
            out[:, np.asarray(hp, dtype=np.int64)] += np.abs(oracle_np.widen(hpv).astype(np.float64))
    return out


def check_fp32(out: np.ndarray, ref: np.ndarray, abs_sum: np.ndarray, N: int):
    """|out - ref| <= 1e-5 |ref|, or, where the terms cancel, <= N 2^-24 sum|term| (fp32 FMA-chain bound)."""
    err = np.abs(out.astype(np.float64) - ref)
    ok = err <= 1e-5 * np.abs(ref)
    ok |= err <= N * 2.0 ** -24 * abs_sum
    return bool(ok.all()), int((~(err <= 1e-5 * np.abs(ref))).sum())


def _bf16_ordinal(bits: np.ndarray) -> np.ndarray:
    b = bits.astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)


def check_bf16(out_bits: np.ndarray, ref: np.ndarray, abs_sum: np.ndarray, N: int):
    """out is bf16_rne(ref) or an adjacent BF16 value; cancellation clause as for fp32."""
    want = torch.from_numpy(ref).to(torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    d = np.abs(_bf16_ordinal(out_bits) - _bf16_ordinal(want))
    ok = d <= 1
    val = oracle_np.widen(out_bits).astype(np.float64)
    ok |= np.abs(val - ref) <= N * 2.0 ** -24 * abs_sum + 2.0 ** -8 * np.abs(ref)
    return bool(ok.all()), int((d > 0).sum())


def run_sync(t: binding.Tpq, ys, k_expect=None, path=binding.PATH_AUTO, stride_pad=0, check_chain=True):
    """Quantise every shard, dequantise+reduce to both output types, compare with the oracle.
    The context must already hold a feature set.  Returns the payloads (host)."""
    orc = oracle.c()
    N, E, bits = t.N, t.E, t.bits
    T = ys[0].shape[0]
    hp = t.get_features()
    k = len(hp)
    if k_expect is not None:
        assert k == k_expect
    s, inv = t.get_scales()
    t.set_option(binding.TPQ_OPT_KERNEL_PATH, path)
    P = t.payload_bytes(T)
    assert P == orc.payload_bytes(T, E, k, bits)
    payload_bufs, payload_host = [], []
    for i in range(N):
        if stride_pad:
            wide = np.zeros((T, E + stride_pad), np.uint16)
            wide[:, :E] = ys[i]
            wide[:, E:] = 0x7FC0                      # NaN in the gap: must never be read as data
            d = dev_bf16(wide)
            stride = E + stride_pad
        else:
            d = dev_bf16(ys[i])
            stride = E
        whole, view = guarded(P)
        t.quantize_pack(i, d.data_ptr(), T, view.data_ptr(), P, row_stride=stride)
        torch.cuda.synchronize()
        assert t.device_status() == 0
        assert guards_intact(whole, P), "quantize_pack wrote outside the payload"
        got = view.cpu().numpy()
        want = orc.quantize_pack(ys[i], hp, inv[i], bits)
        if not np.array_equal(got, want):
            bad = np.nonzero(got != want)[0]
            raise AssertionError(f"payload of shard {i} differs at {bad.size} bytes, first {bad[:8]} "
                                 f"(lp bytes {orc.lp_bytes(T, E, k, bits)}, total {P})")
        payload_bufs.append((whole, view))
        payload_host.append(want)
    ref, chain = orc.dequant_reduce(payload_host, T, E, hp, s, bits=bits)
    abs_sum = term_abs_sum(payload_host, T, E, hp, s, bits)
    ptrs = [v.data_ptr() for _, v in payload_bufs]
    # FP32 output
    whole, view = guarded(T * E * 4)
    t.dequant_reduce(ptrs, T, view.data_ptr(), binding.TPQ_OUT_FP32)
    torch.cuda.synchronize()
    assert guards_intact(whole, T * E * 4)
    out32 = view.cpu().numpy().view(np.float32).reshape(T, E)
    ok, n_cancel = check_fp32(out32, ref, abs_sum, N)
    assert ok, "FP32 output outside tolerance"
    if check_chain:
        assert bits_equal(out32, chain), "FP32 output differs from the ascending binary32 chain"
    # BF16 output, with a padded output stride
    ostride = E + 8
    whole, view = guarded(T * ostride * 2)
    t.dequant_reduce(ptrs, T, view.data_ptr(), binding.TPQ_OUT_BF16, out_row_stride=ostride)
    torch.cuda.synchronize()
    assert guards_intact(whole, T * ostride * 2)
    o = view.cpu().numpy().view(np.uint16).reshape(T, ostride)
    assert (o[:, E:] == (CANARY | (CANARY << 8))).all(), "dequant_reduce wrote into the stride gap"
    ok, _ = check_bf16(o[:, :E], ref, abs_sum, N)
    assert ok, "BF16 output outside tolerance"
    if check_chain:
        assert np.array_equal(o[:, :E], orc.round_bf16(chain))
    return payload_host
