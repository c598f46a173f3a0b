"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle
on the same seeded inputs.  Integer / byte / index results bit-exact; reduction
outputs within 1e-5 relative (FP32) or 1 BF16 ulp (BF16) of the oracle's FP64 sum."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle  # noqa: E402
from paper_2411_07942_b200 import binding, synth  # noqa: E402

import gpu_util as gu  # noqa: E402
from util import bf16_bits, finite_bf16_patterns  # noqa: E402


@pytest.fixture(scope="module", autouse=True)
def _lib():
    gu.ensure_lib()


def _workload(N, T, E, seed, n_out=3, calib=(3, 8)):
    return synth.Workload("t", N, T, E, 0.6, n_out, 20.0, 200.0, calib[0], calib[1], seed)


def _full_pipeline(w, k, path, stride_pad=0, chunks=None, bits=4):
    orc = oracle.c()
    t = binding.Tpq(w.n_shards, w.features, bits=bits)
    scale = synth.column_scales(w)
    cal = [synth.calibration_np(w, i, scale=scale) for i in range(w.n_shards)]
    m, M = gu.calibrate_both(t, cal, chunks=chunks)
    gm, gM = t.get_ranges(with_R=False)
    assert gu.bits_equal(gm, m) and gu.bits_equal(gM, M), "calibration state differs"
    hp = t.select_features(k)
    R, Rbar = orc.ranges(m, M)
    kk = orc.default_k(w.features) if k < 0 else k
    assert hp.tolist() == orc.select(Rbar, kk).tolist()
    _, _, gR, gRbar = t.get_ranges()
    assert gu.bits_equal(gR, R) and gu.bits_equal(gRbar, Rbar)
    s, inv = orc.params(R, bits)
    gs, ginv = t.get_scales()
    assert gu.bits_equal(gs, s) and gu.bits_equal(ginv, inv)
    ys = [synth.activations_np(w, i, w.tokens, scale=scale) for i in range(w.n_shards)]
    gu.run_sync(t, ys, k_expect=kk, path=path, stride_pad=stride_pad)
    t.close()


def test_tiny_config_end_to_end():
    """BASELINE config 1: N=2, 16 tokens x 256 features, 64 calibration tokens, seed 0."""
    w = synth.WORKLOADS["tiny"]
    _full_pipeline(w, -1, binding.PATH_AUTO)          # k = 4: not a multiple of 8 -> shape-generic kernels
    _full_pipeline(w, 8, binding.PATH_TILED)          # same data with k = 8 through the tiled kernels


@pytest.mark.parametrize("N,T,E,k", [(2, 3, 65, 1), (3, 17, 130, 2), (2, 5, 253, 9), (1, 1, 64, 0), (2, 4, 40, 40),
                                     (4, 9, 24, 0), (2, 1, 8, 3), (5, 33, 100, -1)])
def test_generic_path_odd_shapes(N, T, E, k):
    _full_pipeline(_workload(N, T, E, 100 + E + T), k, binding.PATH_AUTO)


@pytest.mark.parametrize("bits", [2, 3, 5, 6, 7, 8])
@pytest.mark.parametrize("N,T,E,k", [(2, 16, 256, 4), (3, 17, 130, 2), (2, 5, 253, 9), (4, 67, 512, 8), (2, 3, 64, 0),
                                     (8, 33, 1024, 16), (2, 129, 5120, 80), (3, 50, 520, 16)])
def test_other_code_widths(bits, N, T, E, k):
    """Other code widths (Section 4 / Figure 3): b-bit codes, step R/(2^b - 1),
    payloads bit-exact against the oracle (codes straddle bytes and words for b = 3, 5, 6, 7), sums in
    tolerance, bits per value b + (16-b)k/E up to the pad."""
    _full_pipeline(_workload(N, T, E, 19 * E + T + bits), k, binding.PATH_AUTO, bits=bits)
    t = binding.Tpq(N, E, bits=bits)
    assert binding.payload_bytes_for(T, E, k, bits) == oracle.c().payload_bytes(T, E, k, bits)
    t.close()


@pytest.mark.parametrize("bits", [2, 3, 5, 6, 7, 8])
def test_other_code_widths_group_kernels_equal_generic(bits):
    """The group kernels (shapes that are multiples of 8) against the oracle and, bit for bit, against the
    shape-generic kernels: strided input, clustered feature sets (several holes in a group, whole groups,
    selected features at the end)."""
    N, T, E = 3, 37, 512
    w = _workload(N, T, E, 90 + bits, calib=(2, 8))
    scale = synth.column_scales(w)
    cal = [synth.calibration_np(w, i, scale=scale) for i in range(N)]
    ys = [synth.activations_np(w, i, T, scale=scale) for i in range(N)]
    rng = np.random.default_rng(bits)
    sets = [list(range(0, 8)), list(range(0, 15)) + [511], list(range(3, 3 + 24)),
            sorted(rng.permutation(E)[:64].tolist()), list(range(E - 8, E)), list(range(8, E)), []]
    for hp in sets:
        t = binding.Tpq(N, E, bits=bits)
        gu.calibrate_both(t, cal)
        t.set_features(hp)
        a = gu.run_sync(t, ys, path=binding.PATH_GENERIC)
        b = gu.run_sync(t, ys, path=binding.PATH_TILED, stride_pad=16)
        for x, y in zip(a, b):
            assert np.array_equal(x, y)
        t.close()


@pytest.mark.parametrize("N,T,E,k,pad", [(2, 67, 512, 8, 0), (4, 301, 1024, 16, 0), (4, 37, 5120, 80, 64),
                                         (8, 64, 4608, 72, 0), (16, 33, 2048, 32, 8), (3, 1, 256, 8, 0),
                                         (2, 150, 8192, 128, 0), (2, 600, 64, 8, 0), (2, 19, 16, 8, 0),
                                         (2, 7, 10240, 160, 0), (4, 12, 256, 0, 0), (2, 11, 256, 248, 0)])
def test_tiled_path_shapes(N, T, E, k, pad):
    """Several tiles, ragged tails, strided input, every group-of-8 hole pattern."""
    _full_pipeline(_workload(N, T, E, 7 * E + T), k, binding.PATH_TILED, stride_pad=pad)


@pytest.mark.parametrize("N,T,E,k", [(10, 2390, 1024, 32), (16, 1203, 2048, 32), (9, 2401, 1024, 0), (13, 2369, 1024, 64),
                                     (2, 1195, 8192, 128)])
def test_tensor_map_panel_kernel_shapes(N, T, E, k):
    """Shapes that dequant_reduce serves with tiled tensor copies (more than 8 devices or long rows, 16-byte
    row pitch, i.e. E - k a multiple of 32, and at least 148 row chunks x panels): device counts that are not a multiple of the 4 devices
    per stage, ragged last chunk, partial last panel, no selected feature at all."""
    _full_pipeline(_workload(N, T, E, 11 * E + T, calib=(2, 8)), k, binding.PATH_TILED)


@pytest.mark.parametrize("N,T,E,k", [(9, 100, 1040, 8), (12, 37, 5120, 80), (33, 21, 1024, 16), (64, 9, 512, 8),
                                     (9, 300, 4608, 72)])
def test_copy_ring_panel_kernel_shapes(N, T, E, k):
    """Shapes served by the asynchronous-copy panel kernel: row pitch not a multiple of 16 bytes, more than
    16 devices (narrower panels), short inputs."""
    _full_pipeline(_workload(N, T, E, 13 * E + T, calib=(2, 8)), k, binding.PATH_TILED)


def test_panel_kernels_equal_generic_on_clustered_feature_sets():
    """The panel kernels on arbitrary feature sets: several holes in one group, whole groups, more selected
    features in a panel than the block has threads, selected features at the very end, nearly everything
    selected.  N = 9 keeps the row kernel out; T = 2400 reaches the tensor-map kernel, T = 50 the copy ring."""
    N, E = 9, 1024
    rng = np.random.default_rng(5)
    sets = [                                             # sizes are multiples of 32: 16-byte row pitch
        list(range(0, 32)),
        list(range(0, 31)) + [1023],
        list(range(3, 3 + 32)),
        sorted(rng.permutation(E)[:128].tolist()),
        sorted(rng.permutation(E)[:512].tolist()),
        list(range(E - 32, E)),
        list(range(32, E)),
        [5, 6, 7, 8, 9, 10] + list(range(100, 340, 10)) + [1000, 1001],
        list(range(0, 8)),                               # (these two: pitch not a multiple of 16 bytes)
        list(range(3, 3 + 24)),
    ]
    for T in (2400, 50):
        w = _workload(N, T, E, 31 + T, calib=(2, 8))
        scale = synth.column_scales(w)
        cal = [synth.calibration_np(w, i, scale=scale) for i in range(N)]
        ys = [synth.activations_np(w, i, T, scale=scale) for i in range(N)]
        for hp in sets:
            t = binding.Tpq(N, E)
            gu.calibrate_both(t, cal)
            t.set_features(hp)
            a = gu.run_sync(t, ys, path=binding.PATH_GENERIC)
            b = gu.run_sync(t, ys, path=binding.PATH_TILED)
            for x, y in zip(a, b):
                assert np.array_equal(x, y)
            t.close()


@pytest.mark.parametrize("N,T,E,k,pad", [(4, 1501, 5120, 80, 0), (2, 1999, 1024, 16, 8), (3, 1600, 4608, 72, 0),
                                         (1, 1481, 256, 8, 0), (4, 1537, 512, 0, 0), (2, 1490, 6144, 96, 0)])
def test_row_kernel_shapes(N, T, E, k, pad):
    """Shapes that dequant_reduce serves with the row kernel (at most 4 devices, at least ten rows per SM):
    ragged last stage, odd rows-per-stage alignment classes of (E-k)/8, strided input, no selected feature."""
    _full_pipeline(_workload(N, T, E, 17 * E + T, calib=(2, 8)), k, binding.PATH_TILED, stride_pad=pad)


def test_row_kernel_equals_generic_on_clustered_feature_sets():
    N, T, E = 3, 1500, 512
    w = _workload(N, T, E, 78, calib=(2, 8))
    scale = synth.column_scales(w)
    cal = [synth.calibration_np(w, i, scale=scale) for i in range(N)]
    ys = [synth.activations_np(w, i, T, scale=scale) for i in range(N)]
    rng = np.random.default_rng(2)
    sets = [list(range(0, 8)), list(range(0, 15)) + [511], list(range(3, 3 + 24)),
            sorted(rng.permutation(E)[:64].tolist()), list(range(E - 8, E)), list(range(8, E))]
    for hp in sets:
        t = binding.Tpq(N, E)
        gu.calibrate_both(t, cal)
        t.set_features(hp)
        a = gu.run_sync(t, ys, path=binding.PATH_GENERIC)
        b = gu.run_sync(t, ys, path=binding.PATH_TILED)
        for x, y in zip(a, b):
            assert np.array_equal(x, y)
        t.close()


@pytest.mark.parametrize("N,T,E,k", [(4, 37, 512, 32), (2, 301, 1024, 32), (3, 16, 4096, 64), (4, 2, 256, 0), (1, 65, 6144, 96),
                                     (8, 70, 1056, 32), (5, 33, 4096, 64), (7, 130, 520, 8),
                                     # rows that are not a multiple of 16 bytes long: (E-k)/8 = 630, 129, 131 (mod 4: 2, 1, 3)
                                     (8, 64, 5120, 80), (8, 36, 1048, 16), (3, 40, 1064, 16)])
def test_every_dequant_kernel_gives_the_same_bits(N, T, E, k):
    """The row, tensor-map panel and copy-ring panel kernels forced in turn on shapes that admit all three
    (short inputs included, where the automatic choice would not pick them): FP32 and BF16 outputs are
    bit-identical to the shape-generic kernel's."""
    w = _workload(N, T, E, 23 * E + T, calib=(2, 8))
    scale = synth.column_scales(w)
    t = binding.Tpq(N, E)
    gu.calibrate_both(t, [synth.calibration_np(w, i, scale=scale) for i in range(N)])
    t.select_features(k)
    P = t.payload_bytes(T)
    pls = []
    for i in range(N):
        y = gu.dev_bf16(synth.activations_np(w, i, T, scale=scale))
        buf = torch.empty(P, dtype=torch.uint8, device="cuda")
        t.quantize_pack(i, y.data_ptr(), T, buf.data_ptr(), P)
        pls.append(buf)
    ptrs = [b.data_ptr() for b in pls]
    outs = {}
    for name, path, kern in [("generic", binding.PATH_GENERIC, binding.DQ_AUTO), ("rows", binding.PATH_TILED, binding.DQ_ROWS),
                             ("tensor", binding.PATH_TILED, binding.DQ_TENSOR_PANELS),
                             ("copy", binding.PATH_TILED, binding.DQ_COPY_PANELS)]:
        t.set_option(binding.TPQ_OPT_KERNEL_PATH, path)
        t.set_option(binding.TPQ_OPT_DEQUANT_KERNEL, kern)
        o32 = torch.full((T, E), float("nan"), dtype=torch.float32, device="cuda")
        o16 = torch.full((T, E), float("nan"), dtype=torch.bfloat16, device="cuda")
        t.dequant_reduce(ptrs, T, o32.data_ptr(), binding.TPQ_OUT_FP32)
        t.dequant_reduce(ptrs, T, o16.data_ptr(), binding.TPQ_OUT_BF16)
        torch.cuda.synchronize()
        assert t.device_status() == 0
        outs[name] = (o32.view(torch.int32).cpu().numpy(), o16.view(torch.int16).cpu().numpy())
    for name in ("rows", "tensor", "copy"):
        assert np.array_equal(outs[name][0], outs["generic"][0]), name
        assert np.array_equal(outs[name][1], outs["generic"][1]), name
    # a kernel the shape does not admit is refused, not silently replaced
    t2 = binding.Tpq(9, 512)
    gu.calibrate_both(t2, [synth.calibration_np(_workload(9, 4, 512, 3, calib=(2, 8)), i) for i in range(9)])
    t2.select_features(8)
    t2.set_option(binding.TPQ_OPT_DEQUANT_KERNEL, binding.DQ_ROWS)
    with pytest.raises(binding.TpqError):
        t2.dequant_reduce([pls[0].data_ptr()] * 9, 1, torch.empty((1, 512), dtype=torch.bfloat16, device="cuda").data_ptr())
    # rows that are not a multiple of 16 bytes long: the tensor-map kernel takes whole groups of 2 (or 4) rows, the
    # shape-generic kernel the rest (the payloads of T rows read as T - 1 rows would differ: fresh ones)
    if (E - k) // 8 % 4 != 0 and T > 4:
        T1 = T - 1
        P1 = t.payload_bytes(T1)
        pl1 = []
        for i in range(N):
            y = gu.dev_bf16(synth.activations_np(w, i, T, scale=scale)[:T1])
            buf = torch.empty(P1, dtype=torch.uint8, device="cuda")
            t.quantize_pack(i, y.data_ptr(), T1, buf.data_ptr(), P1)
            pl1.append(buf)
        got = {}
        for name, path, kern in [("generic", binding.PATH_GENERIC, binding.DQ_AUTO), ("tensor", binding.PATH_TILED, binding.DQ_TENSOR_PANELS)]:
            t.set_option(binding.TPQ_OPT_KERNEL_PATH, path)
            t.set_option(binding.TPQ_OPT_DEQUANT_KERNEL, kern)
            o32 = torch.full((T1, E), float("nan"), dtype=torch.float32, device="cuda")
            o16 = torch.full((T1, E), float("nan"), dtype=torch.bfloat16, device="cuda")
            t.dequant_reduce([b.data_ptr() for b in pl1], T1, o32.data_ptr(), binding.TPQ_OUT_FP32)
            t.dequant_reduce([b.data_ptr() for b in pl1], T1, o16.data_ptr(), binding.TPQ_OUT_BF16)
            torch.cuda.synchronize()
            assert t.device_status() == 0
            got[name] = (o32.view(torch.int32).cpu().numpy(), o16.view(torch.int16).cpu().numpy())
        assert np.array_equal(got["tensor"][0], got["generic"][0])
        assert np.array_equal(got["tensor"][1], got["generic"][1])
    t.close()
    t2.close()


@pytest.mark.parametrize("N,T,E,features", [
    (8, 1501, 5120, None),                              # the automatic choice: 630 groups, two-row stages, ragged end
    (6, 4101, 5120, None),                              # four-row stages, ragged end
    (5, 300, 1016, list(range(4, 1016, 64))),           # an odd number of groups (125): the halves differ by one
    (7, 41, 1016, list(range(0, 16))),                  # every hole in the first block's half
    (8, 41, 1016, list(range(992, 1000)) + list(range(1008, 1016))),   # holes in the second half only, selected features among the last k
    (8, 7, 16, list(range(8, 16))),                     # one group: the second block has none
    (6, 133, 1024, list(range(1, 1024, 2))[:400]),      # more selected features than auxiliary threads
    (5, 64, 512, []),                                   # none selected
])
def test_row_kernel_with_two_blocks_per_run(N, T, E, features):
    """5 to 8 devices: two blocks share a run of rows, each decoding half of the groups.  Forced on shapes that
    reach each of its cases; FP32 and BF16 outputs, with and without a bias, bit-identical to the
    shape-generic kernel's; the first shapes also against the oracle through the automatic choice."""
    w = _workload(N, T, E, 29 * E + T, calib=(2, 8))
    if features is None:
        _full_pipeline(w, E // 64, binding.PATH_TILED)
    scale = synth.column_scales(w)
    t = binding.Tpq(N, E)
    gu.calibrate_both(t, [synth.calibration_np(w, i, scale=scale) for i in range(N)])
    if features is None:
        t.select_features(E // 64)
    else:
        t.set_features(features)
    P = t.payload_bytes(T)
    pls = []
    for i in range(N):
        y = gu.dev_bf16(synth.activations_np(w, i, T, scale=scale))
        buf = torch.empty(P, dtype=torch.uint8, device="cuda")
        t.quantize_pack(i, y.data_ptr(), T, buf.data_ptr(), P)
        pls.append(buf)
    ptrs = [b.data_ptr() for b in pls]
    bias = torch.from_numpy(np.random.default_rng(E + T).standard_normal(E).astype(np.float32)).cuda()
    outs = {}
    for name, path, kern in [("generic", binding.PATH_GENERIC, binding.DQ_AUTO), ("rows", binding.PATH_TILED, binding.DQ_ROWS)]:
        t.set_option(binding.TPQ_OPT_KERNEL_PATH, path)
        t.set_option(binding.TPQ_OPT_DEQUANT_KERNEL, kern)
        got = []
        for b in (None, bias.data_ptr()):
            o32 = torch.full((T, E), float("nan"), dtype=torch.float32, device="cuda")
            o16 = torch.full((T, E), float("nan"), dtype=torch.bfloat16, device="cuda")
            t.dequant_reduce(ptrs, T, o32.data_ptr(), binding.TPQ_OUT_FP32, bias_ptr=b)
            t.dequant_reduce(ptrs, T, o16.data_ptr(), binding.TPQ_OUT_BF16, bias_ptr=b)
            torch.cuda.synchronize()
            assert t.device_status() == 0
            got += [o32.view(torch.int32).cpu().numpy(), o16.view(torch.int16).cpu().numpy()]
        outs[name] = got
    for a, b in zip(outs["rows"], outs["generic"]):
        assert np.array_equal(a, b)
    t.close()


@pytest.mark.parametrize("N,T,E,k", [(4, 301, 1024, 16), (16, 1203, 2048, 32), (9, 100, 1040, 8)])
def test_back_to_back_launches_and_graph_replay_give_the_eager_result(N, T, E, k):
    """Calls enqueued back to back on one stream (the kernels start before the one ahead has drained and wait
    for it before touching its data) and the same calls replayed from a CUDA graph give the bits of calls
    separated by synchronisation; a step may overwrite the buffers of the step before."""
    w = _workload(N, T, E, 29 * E + T, calib=(2, 8))
    scale = synth.column_scales(w)
    t = binding.Tpq(N, E)
    gu.calibrate_both(t, [synth.calibration_np(w, i, scale=scale) for i in range(N)])
    t.select_features(k)
    P = t.payload_bytes(T)
    ys = [[gu.dev_bf16(synth.activations_np(w, i, T, scale=scale) ^ np.uint16(0x8000 * v)) for i in range(N)]
          for v in range(2)]                     # two input sets (the second with every sign flipped)
    pls = [torch.empty(P, dtype=torch.uint8, device="cuda") for _ in range(N)]
    out = torch.empty((T, E), dtype=torch.bfloat16, device="cuda")
    ptrs = [p_.data_ptr() for p_ in pls]

    def step(v, stream):
        t.quantize_pack_batch(0, [y.data_ptr() for y in ys[v]], T, ptrs, P, stream=stream)
        t.dequant_reduce(ptrs, T, out.data_ptr(), stream=stream)

    want = []
    for v in range(2):                           # eager, synchronised
        step(v, 0)
        torch.cuda.synchronize()
        want.append(out.view(torch.int16).cpu().numpy().copy())
    assert not np.array_equal(want[0], want[1])
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):                # back to back: payloads and output reused by consecutive steps
        for rep in range(6):
            step(rep & 1, side.cuda_stream)
    torch.cuda.synchronize()
    assert np.array_equal(out.view(torch.int16).cpu().numpy(), want[1])
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        step(1, side.cuda_stream)
        step(0, side.cuda_stream)
    out.zero_()
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert t.device_status() == 0
    assert np.array_equal(out.view(torch.int16).cpu().numpy(), want[0])
    t.close()


@pytest.mark.parametrize("N,T,E,k,bits", [(4, 37, 512, 32, 4), (2, 301, 1024, 32, 4), (3, 150, 4096, 64, 4), (2, 5, 253, 9, 4),
                                          (3, 33, 512, 8, 8), (2, 19, 130, 2, 3), (4, 64, 512, 0, 4)])
def test_bias_is_added_after_the_sum(N, T, E, k, bits):
    """tpq_dequant_reduce_bias (Section 2: f(x) = sum_i f_i(x_i) + b) on every kernel the shape admits:
    FP32 output bit-identical to the oracle's chain fl(acc + b), BF16 output to its rounding; hole, filler and
    selected columns get their own bias."""
    orc = oracle.c()
    w = _workload(N, T, E, 37 * E + T, calib=(2, 8))
    scale = synth.column_scales(w)
    t = binding.Tpq(N, E, bits=bits)
    gu.calibrate_both(t, [synth.calibration_np(w, i, scale=scale) for i in range(N)])
    hp = t.select_features(k)
    s_, inv = t.get_scales()
    P = t.payload_bytes(T)
    ys = [synth.activations_np(w, i, T, scale=scale) for i in range(N)]
    host = [orc.quantize_pack(ys[i], hp, inv[i], bits) for i in range(N)]
    pls = [torch.from_numpy(h).cuda() for h in host]
    ptrs = [b.data_ptr() for b in pls]
    bias = (np.random.default_rng(E + T).normal(0, 1, E) * np.abs(s_).mean(axis=0) * 5).astype(np.float32)
    bias_d = torch.from_numpy(bias).cuda()
    ref, chain = orc.dequant_reduce(host, T, E, hp, s_, bits=bits, bias=bias)
    want16 = orc.round_bf16(chain)
    tiled = E % 8 == 0 and k % 8 == 0
    kernels = [(binding.PATH_GENERIC, binding.DQ_AUTO)]
    if tiled:
        kernels.append((binding.PATH_TILED, binding.DQ_AUTO))
    if tiled and bits == 4:
        kernels += [(binding.PATH_TILED, binding.DQ_COPY_PANELS)]
        if N <= 4:
            kernels.append((binding.PATH_TILED, binding.DQ_ROWS))
        if (E - k) % 32 == 0:
            kernels.append((binding.PATH_TILED, binding.DQ_TENSOR_PANELS))
    for path, kern in kernels:
        t.set_option(binding.TPQ_OPT_KERNEL_PATH, path)
        t.set_option(binding.TPQ_OPT_DEQUANT_KERNEL, kern)
        o32 = torch.full((T, E), float("nan"), dtype=torch.float32, device="cuda")
        o16 = torch.full((T, E), float("nan"), dtype=torch.bfloat16, device="cuda")
        t.dequant_reduce(ptrs, T, o32.data_ptr(), binding.TPQ_OUT_FP32, bias_ptr=bias_d.data_ptr())
        t.dequant_reduce(ptrs, T, o16.data_ptr(), binding.TPQ_OUT_BF16, bias_ptr=bias_d.data_ptr())
        torch.cuda.synchronize()
        assert t.device_status() == 0
        assert gu.bits_equal(o32.cpu().numpy(), chain), (path, kern)
        assert np.array_equal(o16.view(torch.int16).cpu().numpy().view(np.uint16), want16), (path, kern)
    with pytest.raises(binding.TpqError):
        t.dequant_reduce(ptrs, T, o32.data_ptr(), binding.TPQ_OUT_FP32, bias_ptr=bias_d.data_ptr() + 4)
    t.close()


def test_tiled_equals_generic_on_clustered_feature_sets():
    """Arbitrary feature sets (the paper's random-selection baseline and worse):
    runs of adjacent selected features, whole groups of 8, first and last feature."""
    N, T, E = 3, 29, 512
    w = _workload(N, T, E, 77)
    scale = synth.column_scales(w)
    cal = [synth.calibration_np(w, i, scale=scale) for i in range(N)]
    ys = [synth.activations_np(w, i, T, scale=scale) for i in range(N)]
    rng = np.random.default_rng(1)
    sets = [
        list(range(0, 8)),                                   # a whole group
        list(range(0, 15)) + [511],
        [0, 1, 2, 3, 4, 5, 6, 500, 501, 502, 503, 504, 505, 506, 507, 511],
        list(range(3, 3 + 24)),                              # straddles groups
        sorted(rng.permutation(E)[:64].tolist()),            # random baseline, k = E/8
        sorted(rng.permutation(E)[:8].tolist()),
        list(range(E - 8, E)),
        list(range(8, E)),                                   # only the first group is quantised
    ]
    for hp in sets:
        assert len(hp) % 8 == 0
        t = binding.Tpq(N, E)
        gu.calibrate_both(t, cal)
        t.set_features(hp)
        assert t.get_features().tolist() == hp
        a = gu.run_sync(t, ys, path=binding.PATH_GENERIC)
        b = gu.run_sync(t, ys, path=binding.PATH_TILED)
        for x, y in zip(a, b):
            assert np.array_equal(x, y)
        t.close()


@pytest.mark.parametrize("path", [binding.PATH_GENERIC, binding.PATH_TILED])
def test_quantiser_all_bf16_patterns_and_ties(path):
    """Every non-NaN BF16 pattern through the GPU quantiser at several steps, among them
    s = 1 (exact ties) -- bit-exact against the oracle."""
    orc = oracle.c()
    pats = finite_bf16_patterns()
    E = 256
    T = (pats.size + E - 1) // E
    y = np.zeros(T * E, np.uint16)
    y[: pats.size] = pats
    y = y.reshape(T, E)
    steps = np.array([1.0, 0.37, 3.0e-3, 17.25, 2.0 ** -10, 1.0 / 3.0, 123.456, 2.0 ** -23], np.float32)
    N = len(steps)
    t = binding.Tpq(N, E)
    half_range = (steps * np.float32(7.5)).astype(np.float32)          # R = 2 * 7.5 s = 15 s
    M = np.repeat(half_range[:, None], E, axis=1)
    t.set_ranges(-M, M, np.ones(N, np.int64))
    t.set_features([])
    s, inv = t.get_scales()
    os_, oinv = orc.params((2 * M).astype(np.float32))
    assert gu.bits_equal(s, os_) and gu.bits_equal(inv, oinv)
    t.set_option(binding.TPQ_OPT_KERNEL_PATH, path)
    d = gu.dev_bf16(y)
    P = t.payload_bytes(T)
    for i in range(N):
        whole, view = gu.guarded(P)
        t.quantize_pack(i, d.data_ptr(), T, view.data_ptr(), P)
        torch.cuda.synchronize()
        assert np.array_equal(view.cpu().numpy(), orc.quantize_pack(y, np.zeros(0, np.int32), inv[i])), i
        assert gu.guards_intact(whole, P)
    t.close()


@pytest.mark.parametrize("path", [binding.PATH_GENERIC, binding.PATH_TILED])
def test_quantiser_product_is_rounded_before_the_integer_rounding(path):
    """Searched (x, 1/s) pairs whose float32 product is an exact tie although the exact
    product is not: a fused multiply-add in the kernel would give a different code."""
    orc = oracle.c()
    rng = np.random.default_rng(11)
    E = 256
    xs, invs = [], []
    pats = finite_bf16_patterns()
    from util import bf16_value
    vals = bf16_value(pats)
    cand = pats[(vals > 0.9) & (vals < 1.2)]
    while len(xs) < E:
        xb = int(cand[rng.integers(len(cand))])
        x = float(bf16_value(np.array([xb], np.uint16))[0])
        half = rng.integers(0, 7) + 0.5
        i0 = np.float32(half / x)
        for c in (np.nextafter(i0, np.float32(0)), i0, np.nextafter(i0, np.float32(10))):
            exact = np.float64(x) * np.float64(c)
            if float(np.float32(exact)) == half and exact != half:
                xs.append(xb)
                invs.append(np.float32(c))
                break
    xs = np.array(xs[:E], np.uint16)
    invs = np.array(invs[:E], np.float32)
    # ranges that reproduce these reciprocals exactly are not guaranteed; install steps s with fl(1/s) == inv
    s = (np.float32(1.0) / invs).astype(np.float32)
    keep = (np.float32(1.0) / s).astype(np.float32) == invs
    assert keep.sum() > E // 4
    R = (s * np.float32(15.0)).astype(np.float32)
    ok = (R / np.float32(15.0)).astype(np.float32) == s
    keep &= ok
    assert keep.sum() > E // 8
    M = np.where(keep, R / 2, 1.0).astype(np.float32)[None, :]
    t = binding.Tpq(1, E)
    t.set_ranges(-M, M, np.ones(1, np.int64))
    t.set_features([])
    gs, ginv = t.get_scales()
    assert np.array_equal(ginv[0][keep], invs[keep])
    t.set_option(binding.TPQ_OPT_KERNEL_PATH, path)
    y = np.tile(xs[None, :], (4, 1))
    d = gu.dev_bf16(y)
    P = t.payload_bytes(4)
    whole, view = gu.guarded(P)
    t.quantize_pack(0, d.data_ptr(), 4, view.data_ptr(), P)
    torch.cuda.synchronize()
    want = orc.quantize_pack(y, np.zeros(0, np.int32), ginv[0])
    assert np.array_equal(view.cpu().numpy(), want)
    # and those codes are the tie-to-even ones, not the fused ones
    codes, _ = oracle.oracle_np.unpack(want, 4, E, 0)
    assert np.all(codes[0][keep] % 2 == 0)
    t.close()


def test_selected_features_pass_every_pattern_through():
    """All 65 536 BF16 patterns (NaNs, signed zeros, subnormals) in selected columns arrive unchanged."""
    E, T = 64, 1024
    pats = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    y = np.zeros((T, E), np.uint16)
    hp = list(range(8, 16)) + list(range(40, 48))
    y[:, 8:16] = pats[: T * 8].reshape(T, 8)
    y[:, 40:48] = pats[:: -1][: T * 8].reshape(T, 8)
    for off in (0, 8192 * 4):
        yy = y.copy()
        yy[:, 8:16] = np.roll(pats, -off)[: T * 8].reshape(T, 8)
        t = binding.Tpq(1, E)
        M = np.ones((1, E), np.float32)
        t.set_ranges(-M, M, np.ones(1, np.int64))
        t.set_features(hp)
        for path in (binding.PATH_GENERIC, binding.PATH_TILED):
            t.set_option(binding.TPQ_OPT_KERNEL_PATH, path)
            d = gu.dev_bf16(yy)
            P = t.payload_bytes(T)
            whole, view = gu.guarded(P)
            t.quantize_pack(0, d.data_ptr(), T, view.data_ptr(), P)
            torch.cuda.synchronize()
            got = view.cpu().numpy()
            lpb = oracle.c().lp_bytes(T, E, 16)
            assert np.array_equal(got[lpb:].view(np.uint16).reshape(T, 16), yy[:, hp])
        t.close()


def test_calibration_batching_and_resume():
    """One call with n sequences == n calls; state survives get_state / set_state bit for bit."""
    w = _workload(2, 8, 256, 5, calib=(6, 40))
    scale = synth.column_scales(w)
    cal = [synth.calibration_np(w, i, scale=scale) for i in range(2)]
    a = binding.Tpq(2, 256)
    m, M = gu.calibrate_both(a, cal)
    b = binding.Tpq(2, 256)
    gu.calibrate_both(b, cal, chunks=[1, 2, 3])
    assert all(gu.bits_equal(x, y) for x, y in zip(a.get_ranges(with_R=False), b.get_ranges(with_R=False)))
    assert gu.bits_equal(a.get_ranges(with_R=False)[0], m)
    # resume: first 2 sequences, checkpoint, restore in a fresh context, fold the other 4
    c = binding.Tpq(2, 256)
    gu.calibrate_both(c, [x[:2] for x in cal])
    blob = c.get_state()
    d = binding.Tpq(2, 256)
    d.set_state(blob)
    for i in range(2):
        dd = gu.dev_bf16(cal[i][2:])
        d.calibrate_ranges(i, dd.data_ptr(), 4, 40)
    torch.cuda.synchronize()
    assert all(gu.bits_equal(x, y) for x, y in zip(a.get_ranges(with_R=False), d.get_ranges(with_R=False)))
    # a state with a feature set restores the set and the steps
    hp = a.select_features(-1)
    e = binding.Tpq(2, 256)
    e.set_state(a.get_state())
    assert e.get_features().tolist() == hp.tolist()
    assert all(gu.bits_equal(x, y) for x, y in zip(a.get_scales(), e.get_scales()))
    for t in (a, b, c, d, e):
        t.close()


def test_calibration_prefill_sized_sequences():
    """Several row splits and feature chunks of the tiled extremes kernel, and the generic one."""
    orc = oracle.c()
    for (n_seq, S, E) in [(3, 2048, 4608), (2, 517, 520), (2, 300, 1001)]:
        w = synth.Workload("c", 1, 1, E, 0.7, 5, 20.0, 200.0, n_seq, S, 4000 + E)
        cal = synth.calibration_np(w, 0)
        t = binding.Tpq(1, E)
        m, M = gu.calibrate_both(t, [cal])
        gm, gM = t.get_ranges(with_R=False)
        assert gu.bits_equal(gm, m) and gu.bits_equal(gM, M)
        t.close()


def test_calibration_many_sequences_per_call():
    """More sequences in one call than the fold kernel holds side by side (several passes, a ragged last one),
    with E not a multiple of its feature tile, in one call and split over calls with a non-zero count."""
    for (n_seq, S, E) in [(150, 9, 200), (65, 130, 264), (64, 3, 40)]:
        w = synth.Workload("c", 1, 1, E, 0.7, 3, 20.0, 200.0, n_seq, S, 4100 + E)
        cal = synth.calibration_np(w, 0)
        a = binding.Tpq(1, E)
        m, M = gu.calibrate_both(a, [cal])
        gm, gM = a.get_ranges(with_R=False)
        assert gu.bits_equal(gm, m) and gu.bits_equal(gM, M)
        b = binding.Tpq(1, E)
        gu.calibrate_both(b, [cal], chunks=[1, n_seq - 2, 1])
        hm, hM = b.get_ranges(with_R=False)
        assert gu.bits_equal(hm, m) and gu.bits_equal(hM, M)
        a.close()
        b.close()


def test_signed_zero_and_infinity_extremes():
    t = binding.Tpq(1, 8)
    y = np.zeros((1, 4, 8), np.uint16)
    y[0, :, 0] = [0x0000, 0x8000, 0x0000, 0x8000]          # +0 and -0: min -0, max +0
    y[0, :, 1] = [0x7F80, 0x3F80, 0xFF80, 0x0000]          # +inf, 1, -inf, 0
    y[0, :, 2] = [0x0001, 0x8001, 0x0000, 0x8000]          # subnormals
    m, M = gu.calibrate_both(t, [y])
    gm, gM = t.get_ranges(with_R=False)
    assert gu.bits_equal(gm, m) and gu.bits_equal(gM, M)
    assert gm.view(np.uint32)[0, 0] == 0x80000000 and gM.view(np.uint32)[0, 0] == 0
    t.close()


def test_llama_prefill_full_size():
    """BASELINE config 2 at full size (N=4, 2048 x 5120), the launch configuration the benchmark times."""
    w = synth.WORKLOADS["llama13b_prefill"]
    wc = synth.Workload(w.name, w.n_shards, w.tokens, w.features, w.sd, w.n_outliers, w.outlier_lo, w.outlier_hi,
                        3, 256, w.seed)
    _full_pipeline(wc, -1, binding.PATH_AUTO)


@pytest.mark.parametrize("T,batched", [(2048, False), (8192, True)])
def test_large_config_sampled_rows(T, batched):
    """BASELINE config 5 (N = 16, E = 8192, k = 128) at 2048 tokens with one quantize_pack call per shard and
    at the full 8192 tokens in the launch configuration bench.py times (all shards in one batched launch).
    Payload rows and output rows are compared with the oracle on sampled rows (rows are independent)."""
    orc = oracle.c()
    w = synth.WORKLOADS["large"]
    N, E = w.n_shards, w.features
    scale = synth.column_scales(w)
    t = binding.Tpq(N, E)
    cal = [synth.calibration_np(w, i, n_seq=2, tokens=64, scale=scale) for i in range(N)]
    gu.calibrate_both(t, cal)
    hp = t.select_features(-1)
    k = len(hp)
    assert k == 128
    s, inv = t.get_scales()
    P = t.payload_bytes(T)
    L = E - k
    lpb = orc.lp_bytes(T, E, k)
    ys = [synth.activations_torch(w, i, T, "cuda", scale=scale) for i in range(N)]
    bufs = [gu.guarded(P) for _ in range(N)]
    if batched:
        t.quantize_pack_batch(0, [y.data_ptr() for y in ys], T, [v.data_ptr() for _, v in bufs], P)
    else:
        for i in range(N):
            t.quantize_pack(i, ys[i].data_ptr(), T, bufs[i][1].data_ptr(), P)
    out = torch.empty((T, E), dtype=torch.float32, device="cuda")
    t.dequant_reduce([v.data_ptr() for _, v in bufs], T, out.data_ptr(), binding.TPQ_OUT_FP32)
    outb = torch.empty((T, E), dtype=torch.bfloat16, device="cuda")
    t.dequant_reduce([v.data_ptr() for _, v in bufs], T, outb.data_ptr(), binding.TPQ_OUT_BF16)
    torch.cuda.synchronize()
    assert t.device_status() == 0
    rows = sorted(set([0, 1, T - 1, T - 2] + np.random.default_rng(0).integers(0, T, 28).tolist()))
    host = [v.cpu().numpy() for _, v in bufs]
    for whole, _ in bufs:
        assert gu.guards_intact(whole, P)
    for r in rows:
        row_payloads = []
        for i in range(N):
            y_row = ys[i][r: r + 1].view(torch.int16).cpu().numpy().view(np.uint16)
            want = orc.quantize_pack(y_row, hp, inv[i])                  # T = 1 payload of this row
            got_lp = host[i][r * L // 2: (r + 1) * L // 2]
            got_hp = host[i][lpb + r * k * 2: lpb + (r + 1) * k * 2]
            assert np.array_equal(got_lp, want[: L // 2]), (r, i)
            assert np.array_equal(got_hp, want[orc.lp_bytes(1, E, k):]), (r, i)
            row_payloads.append(want)
        ref, chain = orc.dequant_reduce(row_payloads, 1, E, hp, s)
        abs_sum = gu.term_abs_sum(row_payloads, 1, E, hp, s)
        o32 = out[r: r + 1].cpu().numpy()
        ok, _ = gu.check_fp32(o32, ref, abs_sum, N)
        assert ok, r
        assert gu.bits_equal(o32, chain)
        ob = outb[r: r + 1].view(torch.int16).cpu().numpy().view(np.uint16)
        ok, _ = gu.check_bf16(ob, ref, abs_sum, N)
        assert ok, r
    t.close()


@pytest.mark.parametrize("N,T,E,k,path", [(4, 301, 1024, 16, binding.PATH_TILED), (8, 64, 4608, 72, binding.PATH_TILED),
                                          (3, 17, 130, 2, binding.PATH_AUTO), (16, 40, 512, 8, binding.PATH_TILED),
                                          (20, 9, 256, 8, binding.PATH_TILED), (4, 2048, 5120, 80, binding.PATH_AUTO)])
def test_batched_quantize_equals_per_shard_calls(N, T, E, k, path):
    """tpq_quantize_pack_batch writes, for every shard, exactly the payload of tpq_quantize_pack (and of the oracle)."""
    orc = oracle.c()
    w = _workload(N, T, E, 900 + E + N)
    scale = synth.column_scales(w)
    t = binding.Tpq(N, E)
    gu.calibrate_both(t, [synth.calibration_np(w, i, scale=scale) for i in range(N)])
    hp = t.select_features(k)
    _, inv = t.get_scales()
    t.set_option(binding.TPQ_OPT_KERNEL_PATH, path)
    ys = [synth.activations_np(w, i, T, scale=scale) for i in range(N)]
    dev = [gu.dev_bf16(y) for y in ys]
    P = t.payload_bytes(T)
    bufs = [gu.guarded(P) for _ in range(N)]
    t.quantize_pack_batch(0, [d.data_ptr() for d in dev], T, [v.data_ptr() for _, v in bufs], P)
    torch.cuda.synchronize()
    assert t.device_status() == 0
    for i in range(N):
        whole, view = bufs[i]
        assert gu.guards_intact(whole, P)
        assert np.array_equal(view.cpu().numpy(), orc.quantize_pack(ys[i], hp, inv[i])), i
    # a sub-range of shards
    if N >= 3:
        bufs2 = [gu.guarded(P) for _ in range(2)]
        t.quantize_pack_batch(1, [dev[1].data_ptr(), dev[2].data_ptr()], T, [v.data_ptr() for _, v in bufs2], P)
        torch.cuda.synchronize()
        for j in range(2):
            assert np.array_equal(bufs2[j][1].cpu().numpy(), bufs[1 + j][1].cpu().numpy())
    assert t.raw("tpq_quantize_pack_batch", N - 1, 2, None, T, E, None, P, None) == binding.TPQ_ERR_INVALID_ARG
    t.close()
