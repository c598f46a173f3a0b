"""The layer ahead of the synchronisation point fused with the compressor (Section 2: f^(i)(x^(i)) = x^(i) W^(i),
then C^(i)), through the C ABI.

The kernel accumulates in binary32 on the tensor cores, the oracle rounds the exact sum once, so the BF16 partial
sums may differ by one unit in the last place where the sum lies next to a rounding boundary.  What decides the
codes is the BF16 value, so the payload is checked bit for bit against the oracle's quantiser applied to the
kernel's OWN rounded sums (both sides take the decision from the same BF16 value), and those sums against the
exact sums within half a BF16 unit plus the binary32 accumulation bound."""
import numpy as np
import pytest
import torch

import gpu_util as gu
import oracle
from oracle import oracle_np
from paper_2411_07942_b200 import binding
from util import bf16_bits

pytestmark = pytest.mark.gpu


def _ordinal(bits):
    b = bits.astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)


def _setup(N, T, K, E, k, seed):
    rng = np.random.default_rng(seed)
    xs = [bf16_bits(rng.normal(0, 1, (T, K))) for _ in range(N)]
    col_gain = np.exp(rng.normal(0, 0.7, E))                      # feature ranges differ, a few stand out
    col_gain[rng.choice(E, max(k, 1), replace=False)] *= 8.0
    ws = [bf16_bits(rng.normal(0, 1, (E, K)) * (col_gain[:, None] / np.sqrt(K))) for _ in range(N)]
    return xs, ws


@pytest.mark.parametrize("N,T,K,E,k", [(1, 1, 8, 16, 8), (1, 5, 16, 64, 0), (2, 130, 72, 264, 8), (2, 100, 64, 256, 8), (2, 300, 200, 1032, 16), (1, 128, 128, 192, 0),
                                       (2, 517, 1280, 2048, 32), (4, 2048, 3456, 5120, 80)])
def test_fused_layer(N, T, K, E, k):
    orc = oracle.c()
    xs, ws = _setup(N, T, K, E, k, 1000 + T + E)
    shard = N - 1
    x, w = xs[shard], ws[shard]
    y_ref = oracle_np.linear_bf16(x, w)                           # the library matmul keeps the full-size case quick
    if T * K * E <= 2e8:
        assert np.array_equal(y_ref, orc.linear_bf16(x, w))
    # static ranges from the layer's own outputs (every device's), a little tight so that some values clip
    t = binding.Tpq(N, E)
    m = np.zeros((N, E), np.float32)
    M = np.zeros((N, E), np.float32)
    for i in range(N):
        yi = oracle_np.widen(y_ref if i == shard else oracle_np.linear_bf16(xs[i][: min(T, 64)], ws[i]))
        m[i], M[i] = 0.8 * yi.min(axis=0), 0.8 * yi.max(axis=0)
    t.set_ranges(m, M, np.ones(N, np.int64))
    hp = t.select_features(k)
    _, inv = t.get_scales()
    lp = oracle_np.lp_index(E, hp)
    L = E - k
    # the weight rows in slot order
    wd = gu.dev_bf16(w)
    w_slots = torch.zeros((E, K), dtype=torch.int16, device="cuda")
    t.permute_weight(wd.data_ptr(), K, w_slots.data_ptr())
    torch.cuda.synchronize()
    order = np.concatenate([lp, np.asarray(hp, np.int64)]).astype(np.int64)
    assert np.array_equal(w_slots.cpu().numpy().view(np.uint16), w[order])
    # the fused layer, with and without the optional copy of the rounded sums
    xd = gu.dev_bf16(x)
    P = t.payload_bytes(T)
    whole, view = gu.guarded(P)
    ywhole, yview = gu.guarded(T * E * 2)
    t.linear_quantize_pack(shard, xd.data_ptr(), w_slots.data_ptr(), T, K, view.data_ptr(), P, y_slots_ptr=yview.data_ptr())
    torch.cuda.synchronize()
    assert t.device_status() == 0
    assert gu.guards_intact(whole, P) and gu.guards_intact(ywhole, T * E * 2)
    y_slots = yview.cpu().numpy().view(np.uint16).reshape(T, E)
    y_k = np.empty((T, E), np.uint16)
    y_k[:, order] = y_slots
    # |kernel - exact sum| <= half a BF16 unit of the result + the binary32 accumulation bound K 2^-24 sum|x w|
    # (the second term matters only where the terms cancel); and all but a few values ARE the exact rounding
    xf, wf = oracle_np.widen(x).astype(np.float64), oracle_np.widen(w).astype(np.float64)
    exact, abs_sum = xf @ wf.T, np.abs(xf) @ np.abs(wf).T
    half_unit = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(exact), 1e-300))) - 8)
    err = np.abs(oracle_np.widen(y_k).astype(np.float64) - exact)
    assert (err <= half_unit * (1 + 1e-9) + K * 2.0 ** -24 * abs_sum).all(), "partial sums outside the accumulation bound"
    d = np.abs(_ordinal(y_k) - _ordinal(y_ref))
    assert (d > 0).mean() < 0.01, f"{(d > 0).mean():.4f} of the partial sums differ from the exact rounding"
    want = orc.quantize_pack(y_k, hp, inv[shard])
    got = view.cpu().numpy()
    if not np.array_equal(got, want):
        bad = np.nonzero(got != want)[0]
        raise AssertionError(f"payload differs at {bad.size} bytes, first {bad[:8]} (code bytes {orc.lp_bytes(T, E, k)})")
    whole2, view2 = gu.guarded(P)
    t.linear_quantize_pack(shard, xd.data_ptr(), w_slots.data_ptr(), T, K, view2.data_ptr(), P)
    torch.cuda.synchronize()
    assert gu.guards_intact(whole2, P) and np.array_equal(view2.cpu().numpy(), want)
    # and the payload feeds the reduction like any other: the unfused path on the same BF16 sums gives the same bytes
    plain = torch.zeros(P, dtype=torch.uint8, device="cuda")
    t.quantize_pack(shard, gu.dev_bf16(y_k).data_ptr(), T, plain.data_ptr(), P)
    torch.cuda.synchronize()
    assert np.array_equal(plain.cpu().numpy(), want)
    t.close()


def test_fused_layer_argument_checks():
    t = binding.Tpq(1, 256)
    t.set_ranges(-np.ones((1, 256), np.float32), np.ones((1, 256), np.float32), np.ones(1, np.int64))
    x = torch.zeros((16, 64), dtype=torch.int16, device="cuda")
    w = torch.zeros((256, 64), dtype=torch.int16, device="cuda")
    ws = torch.zeros((256, 64), dtype=torch.int16, device="cuda")
    pl = torch.zeros(16 * 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.TpqError) as e:
        t.permute_weight(w.data_ptr(), 64, ws.data_ptr())
    assert e.value.status == binding.TPQ_ERR_BAD_STATE
    t.select_features(8)
    P = t.payload_bytes(16)
    t.permute_weight(w.data_ptr(), 64, ws.data_ptr())
    for kw, status in [(dict(K=60), binding.TPQ_ERR_INVALID_ARG), (dict(cap=P - 1), binding.TPQ_ERR_SIZE),
                       (dict(x=x.data_ptr() + 2), binding.TPQ_ERR_ALIGN), (dict(shard=1), binding.TPQ_ERR_INVALID_ARG)]:
        a = dict(shard=0, x=x.data_ptr(), K=64, cap=P)
        a.update(kw)
        with pytest.raises(binding.TpqError) as e:
            t.linear_quantize_pack(a["shard"], a["x"], ws.data_ptr(), 16, a["K"], pl.data_ptr(), a["cap"])
        assert e.value.status == status
    with pytest.raises(binding.TpqError):
        t.permute_weight(w.data_ptr(), 64, w.data_ptr())
    t3 = binding.Tpq(1, 256, bits=3)
    t3.set_ranges(-np.ones((1, 256), np.float32), np.ones((1, 256), np.float32), np.ones(1, np.int64))
    t3.select_features(8)
    with pytest.raises(binding.TpqError):
        t3.linear_quantize_pack(0, x.data_ptr(), ws.data_ptr(), 16, 64, pl.data_ptr(), 16 * 256)
    torch.cuda.synchronize()
    t.close()
    t3.close()


def test_fused_layer_and_push_on_random_shapes():
    """Seeded random shapes (E, k, K multiples of 8; any T): the fused layer's payload against the oracle's
    quantiser on its own BF16 sums, and the pushing quantiser's three copies of the same payload."""
    orc = oracle.c()
    rng = np.random.default_rng(411)
    for case in range(12):
        E = int(rng.integers(2, 200)) * 8
        k = int(rng.integers(0, max(1, E // 32) + 1)) * 8
        if E - k < 8:
            k = 0
        T, K, N = int(rng.integers(1, 400)), int(rng.integers(1, 60)) * 8, int(rng.integers(1, 4))
        x = bf16_bits(rng.normal(0, 1, (T, K)))
        gain = np.exp(rng.normal(0, 0.7, E))
        w = bf16_bits(rng.normal(0, 1, (E, K)) * (gain[:, None] / np.sqrt(K)))
        y_ref = oracle_np.linear_bf16(x, w)
        yv = oracle_np.widen(y_ref)
        t = binding.Tpq(N, E)
        t.set_ranges(np.tile(0.8 * yv.min(axis=0), (N, 1)), np.tile(0.8 * yv.max(axis=0), (N, 1)), np.ones(N, np.int64))
        hp = t.select_features(k)
        _, inv = t.get_scales()
        order = np.concatenate([oracle_np.lp_index(E, hp), np.asarray(hp, np.int64)]).astype(np.int64)
        shard = N - 1
        ws = torch.zeros((E, K), dtype=torch.int16, device="cuda")
        t.permute_weight(gu.dev_bf16(w).data_ptr(), K, ws.data_ptr())
        P = t.payload_bytes(T)
        whole, view = gu.guarded(P)
        ywhole, yview = gu.guarded(T * E * 2)
        t.linear_quantize_pack(shard, gu.dev_bf16(x).data_ptr(), ws.data_ptr(), T, K, view.data_ptr(), P,
                               y_slots_ptr=yview.data_ptr())
        torch.cuda.synchronize()
        tag = (case, N, T, K, E, k)
        assert t.device_status() == 0, tag
        assert gu.guards_intact(whole, P) and gu.guards_intact(ywhole, T * E * 2), tag
        y_k = np.empty((T, E), np.uint16)
        y_k[:, order] = yview.cpu().numpy().view(np.uint16).reshape(T, E)
        want = orc.quantize_pack(y_k, hp, inv[shard])
        assert np.array_equal(view.cpu().numpy(), want), tag
        assert (y_k != y_ref).mean() < 0.02, tag
        bufs = [gu.guarded(P) for _ in range(3)]
        words = torch.zeros(3, dtype=torch.int32, device="cuda")
        t.quantize_pack_push(shard, gu.dev_bf16(y_k).data_ptr(), T, [v.data_ptr() for _, v in bufs],
                             [words.data_ptr() + 4 * d for d in range(3)], P, 9)
        torch.cuda.synchronize()
        assert t.device_status() == 0, tag
        for wh, v in bufs:
            assert gu.guards_intact(wh, P) and np.array_equal(v.cpu().numpy(), want), tag
        assert bool((words == 9).all()), tag
        t.close()
