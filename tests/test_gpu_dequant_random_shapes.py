"""Seeded random shapes and feature sets through every dequantise kernel.

Each case draws N, E, k, T, a feature set (the selector's, random, one contiguous run, or both ends of the
feature range) and, half of the time, a bias, quantises synthetic activations with the library, and then
forces each dequantise kernel in turn (row, tensor-map panel, copy-ring panel; those the shape does not admit
refuse and are skipped) and the automatic choice.  FP32 and BF16 outputs must be bit-identical to the
shape-generic kernel's (which the parity tests pin to the oracle), the device status clean and the canary
bands around the outputs intact."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2411_07942_b200 import binding, synth  # noqa: E402

import gpu_util as gu  # noqa: E402


@pytest.fixture(scope="module", autouse=True)
def _lib():
    gu.ensure_lib()


def _case(rng, case):
    N = int(rng.choice([1, 2, 3, 4, 5, 6, 7, 8, 8, 9, 12, 16]))
    E = int(rng.integers(2, 800)) * 8
    mode = int(rng.integers(0, 5))
    if mode == 0:
        k = 0
    elif mode == 1:
        k = (E // 64 + 7) // 8 * 8
    else:
        k = int(rng.integers(1, max(2, E // 40))) * 8
    if E - k < 8:
        k = 0
    T = int(rng.choice([1, 2, 3, 5, 17, 63, 64, 130, 257, 600, 1501, 2300, 4099]))
    if N * T * E > 4e7:
        T = max(1, int(4e7 // (N * E)))
    return N, T, E, k, int(rng.integers(0, 4)), bool(rng.integers(0, 2)), 100 + case


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_every_kernel_on_random_shapes(seed):
    rng = np.random.default_rng(seed)
    ran = {"rows": 0, "tensor": 0, "copy": 0}
    for case in range(14):
        N, T, E, k, fm, with_bias, wseed = _case(rng, case)
        w = synth.Workload("random", N, T, E, 0.7, max(1, E // 100), 20.0, 200.0, 2, 8, wseed)
        scale = synth.column_scales(w)
        t = binding.Tpq(N, E)
        gu.calibrate_both(t, [synth.calibration_np(w, i, scale=scale) for i in range(N)])
        if fm == 0 or k == 0:
            t.select_features(k)
        elif fm == 1:
            t.set_features(sorted(rng.permutation(E)[:k].tolist()))
        elif fm == 2:
            s0 = int(rng.integers(0, E - k + 1))
            t.set_features(list(range(s0, s0 + k)))
        else:
            t.set_features(sorted(set(list(range(0, k // 2)) + list(range(E - (k - k // 2), E)))))
        P = t.payload_bytes(T)
        pls = []
        for i in range(N):
            y = gu.dev_bf16(synth.activations_np(w, i, T, scale=scale))
            buf = torch.empty(P, dtype=torch.uint8, device="cuda")
            t.quantize_pack(i, y.data_ptr(), T, buf.data_ptr(), P)
            pls.append(buf)
        ptrs = [b.data_ptr() for b in pls]
        bias = torch.from_numpy(rng.standard_normal(E).astype(np.float32)).cuda() if with_bias else None
        bp = None if bias is None else bias.data_ptr()
        outs = {}
        for name, path, kern in [("generic", binding.PATH_GENERIC, binding.DQ_AUTO), ("auto", binding.PATH_TILED, binding.DQ_AUTO),
                                 ("rows", binding.PATH_TILED, binding.DQ_ROWS), ("tensor", binding.PATH_TILED, binding.DQ_TENSOR_PANELS),
                                 ("copy", binding.PATH_TILED, binding.DQ_COPY_PANELS)]:
            t.set_option(binding.TPQ_OPT_KERNEL_PATH, path)
            t.set_option(binding.TPQ_OPT_DEQUANT_KERNEL, kern)
            whole32, v32 = gu.guarded(T * E * 4)
            whole16, v16 = gu.guarded(T * E * 2)
            try:
                t.dequant_reduce(ptrs, T, v32.data_ptr(), binding.TPQ_OUT_FP32, bias_ptr=bp)
                t.dequant_reduce(ptrs, T, v16.data_ptr(), binding.TPQ_OUT_BF16, bias_ptr=bp)
            except binding.TpqError:
                assert name not in ("generic", "auto")   # only a forced kernel may refuse a shape
                continue
            torch.cuda.synchronize()
            assert t.device_status() == 0, (name, N, T, E, k)
            assert gu.guards_intact(whole32, T * E * 4) and gu.guards_intact(whole16, T * E * 2), (name, N, T, E, k)
            outs[name] = (v32.cpu().numpy().view(np.int32), v16.cpu().numpy().view(np.int16))
            if name in ran:
                ran[name] += 1
        for name in outs:
            assert np.array_equal(outs[name][0], outs["generic"][0]), (name, N, T, E, k, fm)
            assert np.array_equal(outs[name][1], outs["generic"][1]), (name, N, T, E, k, fm)
        t.close()
    assert ran["copy"] >= 10 and ran["tensor"] >= 5 and ran["rows"] >= 3   # the draw reaches every kernel
