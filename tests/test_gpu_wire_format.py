"""The payload's wire format, as include/tpq.h states it, implemented here by hand.

A second implementation written from the header alone must interoperate with the
library: these tests build payloads in plain Python from the header's "Wire
format" paragraph (code stream, nibble order, slot order by hole filling, BF16
block), hand them to tpq_dequant_reduce through the C ABI and compare with sums
formed by hand; and decode the library's own payloads with the same rule.
Nothing here uses the oracle or the library's tables (tpq_get_slot_order is only
compared with the hand-made table).  The bit count is the paper's (Section 4);
the byte order is this library's."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2411_07942_b200 import binding  # noqa: E402

import gpu_util as gu  # noqa: E402


@pytest.fixture(scope="module", autouse=True)
def _lib():
    gu.ensure_lib()


def slot_order_from_header(E, selected):
    """Slot c carries feature c unless c is selected; the i-th selected feature below L = E-k (a hole)
    is filled with the i-th unselected feature at or above L (a filler)."""
    sel = set(selected)
    L = E - len(sel)
    holes = [j for j in range(L) if j in sel]
    fillers = [j for j in range(L, E) if j not in sel]
    assert len(holes) == len(fillers)
    fill = dict(zip(holes, fillers))
    return [fill.get(c, c) for c in range(L)]


def build_payload(codes, hp_bits, E, selected):
    """codes[t][c]: integer code of slot c of token t (-8..7); hp_bits[t][h]: BF16 pattern of the h-th
    selected feature.  Returns the payload bytes."""
    T, L, k = len(codes), E - len(selected), len(selected)
    n = T * L
    lp = bytearray(((n + 1) // 2 + 15) // 16 * 16)
    for t in range(T):
        for c in range(L):
            p = t * L + c
            nib = codes[t][c] & 0xF
            lp[p // 2] |= nib << (4 * (p % 2))
    hp = bytearray()
    for t in range(T):
        for h in range(k):
            hp += int(hp_bits[t][h]).to_bytes(2, "little")
    return bytes(lp) + bytes(hp)


def bf16_of(x: float) -> int:
    """BF16 pattern of a value that BF16 holds exactly."""
    u = int(np.float32(x).view(np.uint32))
    assert u & 0xFFFF == 0
    return u >> 16


@pytest.mark.parametrize("E,selected,N,T", [
    (8, [1, 6], 2, 3),                                   # the header's example: slots carry 0 7 2 3 4 5
    (16, [1, 14], 2, 3),                                 # one hole, one selected feature above L
    (64, [0, 3, 9, 17, 33, 40, 57, 63], 3, 5),           # shape of the tiled kernels (k = 8)
    (1024, list(range(5, 1024, 64)), 4, 70),             # several stages of the row kernel, ragged tail
    (256, list(range(248, 256)), 2, 9),                  # no holes: the selected features are the last k
    (256, list(range(0, 8)), 8, 6),                      # every hole in the first group; panel kernels (N = 8)
])
def test_hand_built_payload_is_decoded(E, selected, N, T):
    rng = np.random.default_rng(E + N + T)
    k, L = len(selected), E - len(selected)
    order = slot_order_from_header(E, selected)
    if E == 8:
        assert order == [0, 7, 2, 3, 4, 5]
    # static parameters with exactly known steps: R = 2 max(-m, M) = 15 * 2^e  ->  s = 2^e
    expo = rng.integers(-3, 3, size=(N, E))
    step = np.ldexp(1.0, expo).astype(np.float32)
    M = (7.5 * step).astype(np.float32)
    t = binding.Tpq(N, E)
    t.set_ranges(-M, M, np.ones(N, np.int64))
    t.set_features(selected)
    s, _ = t.get_scales()
    assert np.array_equal(s, step)
    assert t.get_slot_order().tolist() == order
    # payloads by hand
    codes = rng.integers(-8, 8, size=(N, T, L))
    hp_vals = rng.integers(-64, 64, size=(N, T, k)).astype(np.float64) * 0.25     # exact in BF16, sums exact
    payloads = []
    for i in range(N):
        hp_bits = [[bf16_of(hp_vals[i, tt, h]) for h in range(k)] for tt in range(T)]
        pl = build_payload(codes[i].tolist(), hp_bits, E, selected)
        assert len(pl) == t.payload_bytes(T)
        payloads.append(torch.frombuffer(bytearray(pl), dtype=torch.uint8).cuda())
    # expected sums by hand (every term and every partial sum is exact in binary32)
    want = np.zeros((T, E), np.float64)
    for i in range(N):
        for c, j in enumerate(order):
            want[:, j] += codes[i, :, c] * float(step[i, j])
        for h, j in enumerate(selected):
            want[:, j] += hp_vals[i, :, h]
    out = torch.zeros((T, E), dtype=torch.float32, device="cuda")
    t.dequant_reduce([p.data_ptr() for p in payloads], T, out.data_ptr(), binding.TPQ_OUT_FP32)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy().astype(np.float64), want)
    t.close()


@pytest.mark.parametrize("E,selected,T", [(16, [1, 14], 3), (64, [0, 3, 9, 17, 33, 40, 57, 63], 5),
                                          (1024, list(range(5, 1024, 64)), 37)])
def test_library_payload_is_decoded_by_hand(E, selected, T):
    """tpq_quantize_pack's bytes, taken apart with the header's rule: inputs on the quantiser's grid come
    back exactly, slot by slot, and the selected features' patterns sit in the BF16 block."""
    rng = np.random.default_rng(E + T)
    k, L = len(selected), E - len(selected)
    order = slot_order_from_header(E, selected)
    expo = rng.integers(-3, 3, size=(1, E))
    step = np.ldexp(1.0, expo).astype(np.float32)
    M = (7.5 * step).astype(np.float32)
    t = binding.Tpq(1, E)
    t.set_ranges(-M, M, np.ones(1, np.int64))
    t.set_features(selected)
    q = rng.integers(-8, 8, size=(T, E))
    y = (q * step[0]).astype(np.float32)                    # on the grid: the code of y is q
    yb = (y.view(np.uint32) >> 16).astype(np.uint16)        # exact in BF16 (3 significant bits)
    d = gu.dev_bf16(yb)
    P = t.payload_bytes(T)
    whole, pl = gu.guarded(P)
    t.quantize_pack(0, d.data_ptr(), T, pl.data_ptr(), P)
    torch.cuda.synchronize()
    assert gu.guards_intact(whole, P)
    b = pl.cpu().numpy()
    lp_bytes = ((T * L + 1) // 2 + 15) // 16 * 16
    for tt in range(T):
        for c, j in enumerate(order):
            p = tt * L + c
            nib = (int(b[p // 2]) >> (4 * (p % 2))) & 0xF
            code = nib - 16 if nib >= 8 else nib
            assert code == q[tt, j], (tt, c, j)
    assert not b[(T * L + 1) // 2: lp_bytes].any()          # padding
    if T * L % 2:
        assert int(b[T * L // 2]) >> 4 == 0
    hp = b[lp_bytes:].view(np.uint16).reshape(T, k)
    assert np.array_equal(hp, yb[:, selected])
    t.close()
