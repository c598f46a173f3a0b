"""The fused exchange (Section 5: all-gather, then a local reduction) through the C ABI on one GPU.

A pushing quantiser stores its payload into several destinations and publishes arrival words; the reducing side
waits for the words with a limit.  With one GPU the N ranks are emulated in ONE stream (every wait is enqueued
behind the pushes it waits for, so nothing ever waits for a kernel that is not already done); the destinations
are plain local buffers, exactly what a peer-mapped pointer is to the kernel."""
import numpy as np
import pytest
import torch

import gpu_util as gu
import oracle
from paper_2411_07942_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _ctx(N, T, E, k, bits=4, seed=0):
    w = synth.Workload("x", N, T, E, 0.7, 5, 20.0, 200.0, 2, 8, 7000 + seed + E + T)
    scale = synth.column_scales(w)
    t = binding.Tpq(N, E, bits=bits)
    gu.calibrate_both(t, [synth.calibration_np(w, i, scale=scale) for i in range(N)])
    hp = t.select_features(k)
    ys = [synth.activations_np(w, i, T, scale=scale) for i in range(N)]
    return t, hp, ys


def _words(n):
    """n arrival words inside a canary-filled int32 tensor; returns (tensor, index of the first word)."""
    pad = 16
    f = torch.full((n + 2 * pad,), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    f[pad: pad + n] = 0
    return f, pad


@pytest.mark.parametrize("N,T,E,k,bits,n_dst", [(2, 301, 1024, 16, 4, 3), (4, 2048, 5120, 80, 4, 4), (2, 37, 512, 0, 4, 1),
                                                (2, 5, 253, 9, 4, 2), (2, 33, 512, 8, 3, 3), (2, 64, 8192, 128, 4, 16)])
def test_push_writes_every_destination_and_publishes(N, T, E, k, bits, n_dst):
    orc = oracle.c()
    t, hp, ys = _ctx(N, T, E, k, bits)
    _, inv = t.get_scales()
    P = t.payload_bytes(T)
    shard = N - 1
    want = orc.quantize_pack(ys[shard], hp, inv[shard], bits)
    y = gu.dev_bf16(ys[shard])
    bufs = [gu.guarded(P) for _ in range(n_dst)]
    f, f0 = _words(n_dst)
    for epoch in (5, 6, 0xFFFFFFFF):      # launches back to back: the block counter returns to zero by itself
        for _, v in bufs:
            v.fill_(0x33)
        t.quantize_pack_push(shard, y.data_ptr(), T, [v.data_ptr() for _, v in bufs],
                             [f.data_ptr() + 4 * (f0 + d) for d in range(n_dst)], P, epoch)
        torch.cuda.synchronize()
        assert t.device_status() == 0
        for d, (whole, v) in enumerate(bufs):
            assert gu.guards_intact(whole, P), f"destination {d}: wrote outside the payload"
            assert np.array_equal(v.cpu().numpy(), want), f"destination {d} differs from the oracle's payload"
        fh = f.cpu().numpy().view(np.uint32)
        assert (fh[f0: f0 + n_dst] == epoch).all()
        assert (fh[:f0] == 0x5A5A5A5A).all() and (fh[f0 + n_dst:] == 0x5A5A5A5A).all()
    t.close()


@pytest.mark.parametrize("N,T,E,k", [(4, 150, 1024, 16), (2, 2048, 5120, 80), (8, 64, 2048, 32)])
def test_emulated_ranks_exchange_and_reduce(N, T, E, k):
    """Every rank pushes its shard into its slot of every rank's receive buffer; every rank waits for its N
    arrival words and reduces its own buffer: all N outputs are the oracle's sum.  Two slot sets alternate."""
    orc = oracle.c()
    t, hp, ys = _ctx(N, T, E, k)
    s, inv = t.get_scales()
    P = t.payload_bytes(T)
    Pa = (P + 255) // 256 * 256
    host = [orc.quantize_pack(ys[i], hp, inv[i]) for i in range(N)]
    _, chain = orc.dequant_reduce(host, T, E, hp, s)
    want16 = orc.round_bf16(chain)
    yd = [gu.dev_bf16(y) for y in ys]
    recv = [torch.zeros(2 * N * Pa, dtype=torch.uint8, device="cuda") for _ in range(N)]     # [set][slot] per rank
    flags = [torch.zeros(2 * N, dtype=torch.int32, device="cuda") for _ in range(N)]
    outs = [torch.full((T, E), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(N)]
    for epoch in (1, 2, 3):
        st = epoch & 1
        for o in outs:
            o.fill_(float("nan"))
        for r in range(N):   # rank r's push
            t.quantize_pack_push(r, yd[r].data_ptr(), T,
                                 [recv[p].data_ptr() + (st * N + r) * Pa for p in range(N)],
                                 [flags[p].data_ptr() + 4 * (st * N + r) for p in range(N)], P, epoch)
        for p in range(N):   # rank p's wait and local reduction: the wait as a launch of its own, or in the reduction
            slots = [recv[p].data_ptr() + (st * N + r) * Pa for r in range(N)]
            if (epoch + p) & 1:
                t.wait_arrivals(flags[p].data_ptr() + 4 * st * N, N, epoch, timeout_ns=200_000_000)
                t.dequant_reduce(slots, T, outs[p].data_ptr(), binding.TPQ_OUT_BF16)
            else:
                t.dequant_reduce(slots, T, outs[p].data_ptr(), binding.TPQ_OUT_BF16,
                                 arrived_ptr=flags[p].data_ptr() + 4 * st * N, epoch=epoch, timeout_ns=200_000_000)
        torch.cuda.synchronize()
        assert t.device_status() == 0
        for p in range(N):
            assert np.array_equal(outs[p].view(torch.int16).cpu().numpy().view(np.uint16), want16), (epoch, p)
    t.close()


def test_wait_gives_up_and_the_context_stays_usable():
    """An arrival word that nothing writes: the wait returns after its limit with TPQ_ERR_TIMEOUT in the device
    status; the next step on the same context runs normally."""
    t, hp, ys = _ctx(2, 19, 512, 8)
    f = torch.zeros(2, dtype=torch.int32, device="cuda")
    f[0] = 9
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    t.wait_arrivals(f.data_ptr(), 2, 9, timeout_ns=20_000_000)
    ev1.record()
    torch.cuda.synchronize()
    assert 15.0 < ev0.elapsed_time(ev1) < 500.0
    assert t.device_status() == binding.TPQ_ERR_TIMEOUT
    assert t.device_status() == 0          # reading clears it
    f[1] = 9
    t.wait_arrivals(f.data_ptr(), 2, 9, timeout_ns=20_000_000)
    torch.cuda.synchronize()
    assert t.device_status() == 0
    gu.run_sync(t, ys, k_expect=8)
    t.close()


@pytest.mark.parametrize("N,T,E,k,bits", [(2, 40, 1024, 32, 4), (2, 9, 253, 9, 4), (2, 33, 512, 8, 3)])
def test_reduction_with_its_own_wait_on_every_kernel(N, T, E, k, bits):
    """tpq_dequant_reduce_arrivals on every kernel the shape admits: with the words set the output (bias included)
    is bit-identical to the plain call's; with a word that nothing writes every block gives up after the limit
    and the status says so."""
    orc = oracle.c()
    t, hp, ys = _ctx(N, T, E, k, bits)
    s_, inv = t.get_scales()
    host = [orc.quantize_pack(ys[i], hp, inv[i], bits) for i in range(N)]
    pls = [torch.from_numpy(h).cuda() for h in host]
    ptrs = [b.data_ptr() for b in pls]
    bias = (np.random.default_rng(E).normal(0, 1, E) * np.abs(s_).mean(axis=0) * 5).astype(np.float32)
    bias_d = torch.from_numpy(bias).cuda()
    _, chain = orc.dequant_reduce(host, T, E, hp, s_, bits=bits, bias=bias)
    tiled = E % 8 == 0 and k % 8 == 0
    kernels = [(binding.PATH_GENERIC, binding.DQ_AUTO)]
    if tiled:
        kernels.append((binding.PATH_TILED, binding.DQ_AUTO))
    if tiled and bits == 4:
        kernels += [(binding.PATH_TILED, binding.DQ_COPY_PANELS), (binding.PATH_TILED, binding.DQ_ROWS)]
        if (E - k) % 32 == 0:
            kernels.append((binding.PATH_TILED, binding.DQ_TENSOR_PANELS))
    words = torch.zeros(N, dtype=torch.int32, device="cuda")
    for path, kern in kernels:
        t.set_option(binding.TPQ_OPT_KERNEL_PATH, path)
        t.set_option(binding.TPQ_OPT_DEQUANT_KERNEL, kern)
        words.fill_(77)
        o32 = torch.full((T, E), float("nan"), dtype=torch.float32, device="cuda")
        t.dequant_reduce(ptrs, T, o32.data_ptr(), binding.TPQ_OUT_FP32, bias_ptr=bias_d.data_ptr(),
                         arrived_ptr=words.data_ptr(), epoch=77, timeout_ns=100_000_000)
        torch.cuda.synchronize()
        assert t.device_status() == 0
        assert gu.bits_equal(o32.cpu().numpy(), chain), (path, kern)
        words[N - 1] = 76                       # the last device's payload "has not arrived"
        t.dequant_reduce(ptrs, T, o32.data_ptr(), binding.TPQ_OUT_FP32, arrived_ptr=words.data_ptr(), epoch=77,
                         timeout_ns=3_000_000)
        torch.cuda.synchronize()
        assert t.device_status() == binding.TPQ_ERR_TIMEOUT, (path, kern)
    t.set_option(binding.TPQ_OPT_KERNEL_PATH, binding.PATH_AUTO)
    t.set_option(binding.TPQ_OPT_DEQUANT_KERNEL, binding.DQ_AUTO)
    gu.run_sync(t, ys, k_expect=k)              # and the context is as usable as before
    t.close()


def test_push_argument_checks():
    t, hp, ys = _ctx(2, 19, 512, 8)
    P = t.payload_bytes(19)
    y = gu.dev_bf16(ys[0])
    buf = torch.zeros(P + 64, dtype=torch.uint8, device="cuda")
    f = torch.zeros(4, dtype=torch.int32, device="cuda")
    ok = dict(dst_ptrs=[buf.data_ptr()], arrived_ptrs=[f.data_ptr()], dst_capacity=P, epoch=1)

    def bad(status, **kw):
        a = dict(ok, **kw)
        with pytest.raises(binding.TpqError) as e:
            t.quantize_pack_push(kw.pop("shard", 0), y.data_ptr(), kw.pop("T", 19), a["dst_ptrs"], a["arrived_ptrs"],
                                 a["dst_capacity"], a["epoch"])
        assert e.value.status == status

    bad(binding.TPQ_ERR_SIZE, dst_capacity=P - 1)
    bad(binding.TPQ_ERR_ALIGN, dst_ptrs=[buf.data_ptr() + 8])
    bad(binding.TPQ_ERR_ALIGN, arrived_ptrs=[f.data_ptr() + 2])
    bad(binding.TPQ_ERR_INVALID_ARG, dst_ptrs=[buf.data_ptr()] * 17, arrived_ptrs=[f.data_ptr()] * 17)
    bad(binding.TPQ_ERR_INVALID_ARG, dst_ptrs=[], arrived_ptrs=[])
    bad(binding.TPQ_ERR_INVALID_ARG, shard=2)
    bad(binding.TPQ_ERR_INVALID_ARG, T=0)
    with pytest.raises(binding.TpqError):
        t.wait_arrivals(f.data_ptr(), 0, 1)
    with pytest.raises(binding.TpqError):
        t.wait_arrivals(f.data_ptr(), 2, 1, timeout_ns=6_000_000_000)
    with pytest.raises(binding.TpqError):
        t.wait_arrivals(f.data_ptr() + 2, 2, 1)
    torch.cuda.synchronize()
    assert t.device_status() == 0
    t.close()


def test_exchange_classes_with_one_rank():
    """The Python exchange layer with a single rank (no process group): both forms give the oracle's output of
    the one shard, step after step on alternating slot sets."""
    from paper_2411_07942_b200.exchange import AllGatherExchange, PushExchange

    orc = oracle.c()
    T, E, k = 77, 1024, 16
    t, hp, _ = _ctx(1, T, E, k)
    s, inv = t.get_scales()
    w = synth.Workload("x", 1, T, E, 0.7, 5, 20.0, 200.0, 2, 8, 4242)
    push = PushExchange(t, T, timeout_ns=100_000_000)
    gather = AllGatherExchange(t.payload_bytes(T))
    scratch = torch.zeros(t.payload_bytes(T), dtype=torch.uint8, device="cuda")
    for step in range(4):
        y = synth.activations_np(synth.Workload("x", 1, T, E, 0.7, 5, 20.0, 200.0, 2, 8, 4242 + step), 0, T)
        yd = gu.dev_bf16(y)
        want = orc.round_bf16(orc.dequant_reduce([orc.quantize_pack(y, hp, inv[0])], T, E, hp, s)[1])
        for ex in ("push", "gather"):
            out = torch.full((T, E), float("nan"), dtype=torch.bfloat16, device="cuda")
            if ex == "push":
                push.step(yd.data_ptr(), out.data_ptr(), binding.TPQ_OUT_BF16)
            else:
                gather.step(t, yd.data_ptr(), T, out.data_ptr(), binding.TPQ_OUT_BF16, scratch)
            torch.cuda.synchronize()
            assert t.device_status() == 0
            assert np.array_equal(out.view(torch.int16).cpu().numpy().view(np.uint16), want), (step, ex)
    assert push.step_no == 4
    t.close()
