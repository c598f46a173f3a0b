"""Host logic of the exchange between ranks (Section 5: all-gather, then a local reduction) on CPU.

World-size-2 gloo ranks: every rank runs the whole path of its own shard with the oracle standing in for the
GPU kernels, exchanges the payload bytes and the calibration rows through the package's exchange layer, and
must end with the oracle's synchronised sum.  The receive-buffer layout of the fused (push) form is pure
arithmetic and is checked directly."""
import json
import os
import socket
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

WORKER = r"""
import os, sys, json
sys.path.insert(0, sys.argv[1])
import numpy as np, torch
import torch.distributed as dist
import oracle
from paper_2411_07942_b200 import synth
from paper_2411_07942_b200.exchange import AllGatherExchange, gather_rows

rank = int(os.environ["RANK"])
dist.init_process_group("gloo", init_method="env://")
N, T, E, k = 2, 21, 256, 4
orc = oracle.c()
w = synth.Workload("x", N, T, E, 0.7, 5, 20.0, 200.0, 3, 16, 991)
scale = synth.column_scales(w)
# rank r calibrates its own shard only, then the rows are shared
m, M, cnt = orc.calibrate(None, None, 0, synth.calibration_np(w, rank, scale=scale), 0.01)
rows = gather_rows(np.concatenate([m, M]).astype(np.float32))
counts = gather_rows(np.asarray([cnt], dtype=np.int64)).reshape(N)
m_all, M_all = rows[:, :E], rows[:, E:]
R, Rbar = orc.ranges(m_all, M_all)
hp = orc.select(Rbar, k)
s, inv = orc.params(R)
y = synth.activations_np(w, rank, T, scale=scale)
mine = orc.quantize_pack(y, hp, inv[rank])
ex = AllGatherExchange(mine.size)
allp = ex.gather(torch.from_numpy(mine.copy())).numpy()
ref, chain = orc.dequant_reduce([allp[i] for i in range(N)], T, E, hp, s)
# what a single process computes from all shards
ms, Ms = zip(*[orc.calibrate(None, None, 0, synth.calibration_np(w, i, scale=scale), 0.01)[:2] for i in range(N)])
R1, Rbar1 = orc.ranges(np.stack(ms), np.stack(Ms))
hp1 = orc.select(Rbar1, k)
s1, inv1 = orc.params(R1)
pl1 = [orc.quantize_pack(synth.activations_np(w, i, T, scale=scale), hp1, inv1[i]) for i in range(N)]
ref1, chain1 = orc.dequant_reduce(pl1, T, E, hp1, s1)
print(json.dumps({"rank": rank, "counts": counts.tolist(), "hp_equal": hp.tolist() == hp1.tolist(),
                  "payloads_equal": all(np.array_equal(allp[i], pl1[i]) for i in range(N)),
                  "sum_equal": bool(np.array_equal(chain.view(np.uint32), chain1.view(np.uint32)))}))
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_exchange_rows_and_payloads(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err
        o = json.loads(out.strip().splitlines()[-1])
        assert o["counts"] == [3, 3]
        assert o["hp_equal"] and o["payloads_equal"] and o["sum_equal"], o


def test_single_process_gather_is_the_identity():
    import torch
    from paper_2411_07942_b200.exchange import AllGatherExchange, gather_rows

    row = np.arange(6, dtype=np.float32)
    assert np.array_equal(gather_rows(row), row[None])
    p = torch.arange(32, dtype=torch.uint8)
    assert torch.equal(AllGatherExchange(32).gather(p), p[None])


def test_receive_layout():
    from paper_2411_07942_b200.exchange import ReceiveLayout

    L = ReceiveLayout(4, 5488640)
    assert L.slot_bytes % 256 == 0 and L.slot_bytes >= 5488640
    spans = []
    for step in (0, 1):
        for r in range(4):
            spans.append((L.slot(step, r), L.slot(step, r) + L.payload_bytes))
            assert L.slot(step, r) % 16 == 0 and L.word(step, r) % 4 == 0
    spans.sort()
    assert all(a[1] <= b[0] for a, b in zip(spans, spans[1:]))          # slots do not overlap
    words = sorted(L.word(s, r) for s in (0, 1) for r in range(4))
    assert words[0] >= spans[-1][1] and len(set(words)) == 8 and words[-1] + 4 <= L.total_bytes
    assert [L.word(0, r) for r in range(4)] == list(range(L.words_offset, L.words_offset + 16, 4))  # one wait covers N words
    # the two steps that share a slot set carry different tags, and no tag is 0 (a zeroed buffer never matches)
    assert L.slot(5, 2) == L.slot(7, 2) and L.slot(5, 2) != L.slot(6, 2)
    for s in (0, 1, 2, 0x7FFFFFFE, 0x7FFFFFFF, 2 ** 40 + 3):
        assert 1 <= L.epoch(s) <= 0xFFFFFFFF
        assert L.epoch(s) != L.epoch(s + 2)


class _FakeRanks:
    """N ranks' receive buffers as host byte arrays behind made-up addresses, and a stand-in for the
    library context that carries out a push and a reduction on them the way the kernels do: a push stores
    the payload at every destination and then the tag in every arrival word; a reduction first checks
    that its N words carry the tag, then reads its N slots."""

    def __init__(self, world, payload_bytes, total_bytes):
        self.world, self.P = world, payload_bytes
        # rank q reaches rank p's buffer at base[q][p]: every rank has its own view of every peer
        self.base = [[0x100000000 * (q + 1) + 0x1000000 * p for p in range(world)] for q in range(world)]
        self.mem = [bytearray(total_bytes) for _ in range(world)]
        self.log = []

    def resolve(self, viewer, addr):
        for p in range(self.world):
            off = addr - self.base[viewer][p]
            if 0 <= off < len(self.mem[p]):
                return p, off
        raise AssertionError(f"rank {viewer} used an address outside every mapped buffer: {addr:#x}")

    def context(self, rank):
        ranks = self

        class Ctx:
            N = ranks.world

            def payload_bytes(self, T):
                return ranks.P

            def quantize_pack_push(self, shard, y_ptr, T, dst, words, cap, epoch, stream=0):
                assert shard == rank and len(dst) == len(words) == ranks.world and cap >= ranks.P
                payload = bytes([(y_ptr + shard) & 0xFF]) * ranks.P        # y_ptr stands for the step's data
                for p in range(ranks.world):
                    owner, off = ranks.resolve(rank, dst[p])
                    assert owner == p, "destination p must be rank p's buffer"
                    ranks.mem[p][off: off + ranks.P] = payload
                for p in range(ranks.world):
                    owner, off = ranks.resolve(rank, words[p])
                    assert owner == p
                    ranks.mem[p][off: off + 4] = int(epoch).to_bytes(4, "little")
                ranks.log.append(("push", rank, epoch))

            def dequant_reduce(self, payloads, T, out_ptr, out_dtype, stream=0, bias_ptr=None, arrived_ptr=None,
                               epoch=0, timeout_ns=0):
                assert len(payloads) == ranks.world and arrived_ptr is not None and timeout_ns > 0
                owner, woff = ranks.resolve(rank, arrived_ptr)
                assert owner == rank, "a reduction waits on words in its own buffer"
                got = []
                for i in range(ranks.world):
                    word = int.from_bytes(ranks.mem[rank][woff + 4 * i: woff + 4 * i + 4], "little")
                    assert word == epoch, f"rank {rank} would wait for ever: word {i} is {word}, tag {epoch}"
                    owner, off = ranks.resolve(rank, payloads[i])
                    assert owner == rank, "a reduction reads local memory only"
                    blob = ranks.mem[rank][off: off + ranks.P]
                    assert len(set(blob)) == 1
                    got.append(blob[0])
                ranks.log.append(("reduce", rank, epoch, tuple(got)))

        return Ctx()


def test_push_exchange_bookkeeping_for_several_ranks():
    """world = 2 and 4, several steps on alternating slot sets: rank r writes slot r of every peer, the
    reductions find the step's payloads of all ranks in their own buffer, tags differ between the steps that
    share a set.  (The symmetric-memory rendezvous itself needs several GPUs and is not exercised here.)"""
    from paper_2411_07942_b200.exchange import PeerBuffers, PushExchange, ReceiveLayout

    for world in (2, 4):
        P = 1000 + 16 * world
        L = ReceiveLayout(world, P)
        ranks = _FakeRanks(world, P, L.total_bytes)
        ex = [PushExchange(ranks.context(r), 7, buffers=PeerBuffers(r, ranks.base[r]), timeout_ns=10 ** 6)
              for r in range(world)]
        for step in range(5):
            # every rank pushes (in any order), then every rank reduces: what one stream per GPU does, given
            # that a reduction waits for the N arrivals
            for r in reversed(range(world)):
                dst, words, tag = ex[r].push_args(step)
                assert tag == L.epoch(step) and len(set(dst)) == world
                assert [ranks.resolve(r, d) for d in dst] == [(p, L.slot(step, r)) for p in range(world)]
                assert [ranks.resolve(r, a) for a in words] == [(p, L.word(step, r)) for p in range(world)]
            for r in range(world):
                # the "data" of rank r in this step is 10 * step (+ r, added by the stand-in)
                ctx = ex[r].tpq
                dst, words, tag = ex[r].push_args(step)
                ctx.quantize_pack_push(r, 10 * step, 7, dst, words, L.slot_bytes, tag)
            for r in range(world):
                payloads, first_word, tag = ex[r].reduce_args(step)
                ex[r].tpq.dequant_reduce(payloads, 7, 0, 0, arrived_ptr=first_word, epoch=tag, timeout_ns=10 ** 6)
                ex[r].step_no += 1
            reduces = [e for e in ranks.log if e[0] == "reduce" and e[2] == L.epoch(step)]
            assert len(reduces) == world
            for e in reduces:
                assert e[3] == tuple((10 * step + i) & 0xFF for i in range(world)), "a rank read another step's payload"
        # step() itself issues the same two calls
        ranks.log.clear()
        for r in range(world):
            ex[r].tpq.quantize_pack_push(r, 77, 7, *ex[r].push_args(ex[r].step_no)[:2], L.slot_bytes,
                                         ex[r].push_args(ex[r].step_no)[2])
        before = [e.step_no for e in ex]
        for r in range(world):
            ex[r].step(77, 0, 0)
        assert [e.step_no for e in ex] == [b + 1 for b in before]
        assert [e[0] for e in ranks.log].count("reduce") == world


def test_push_exchange_rejects_a_wrong_world():
    import pytest
    from paper_2411_07942_b200.exchange import PeerBuffers, PushExchange

    ranks = _FakeRanks(2, 64, 4096)
    with pytest.raises(ValueError):
        PushExchange(ranks.context(0), 7, buffers=PeerBuffers(0, [1, 2, 3]))      # 3 mappings, context of 2 shards


SHARE_WORKER = r"""
import os, sys, json
sys.path.insert(0, sys.argv[1])
import numpy as np, torch
import torch.distributed as dist
from paper_2411_07942_b200.exchange import share_ranges

rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo", init_method="env://")
E = 40

class Ctx:                      # the part of the library context that share_ranges uses
    N, E = world, 40
    def __init__(self):
        self.m = np.zeros((world, E), np.float32); self.M = np.zeros((world, E), np.float32); self.cnt = None
        self.m[rank] = -(rank + 1) * np.arange(1, E + 1, dtype=np.float32)        # only the own row is calibrated
        self.M[rank] = (rank + 1) * np.arange(1, E + 1, dtype=np.float32) + 0.5
    def get_ranges(self, with_R=True):
        return self.m.copy(), self.M.copy()
    def set_ranges(self, m, M, counts):
        self.m, self.M, self.cnt = np.array(m), np.array(M), np.array(counts)

c = Ctx()
share_ranges(c, 3 + rank)
want_m = np.stack([-(r + 1) * np.arange(1, E + 1, dtype=np.float32) for r in range(world)])
want_M = np.stack([(r + 1) * np.arange(1, E + 1, dtype=np.float32) + 0.5 for r in range(world)])
print(json.dumps({"ok": bool(np.array_equal(c.m, want_m) and np.array_equal(c.M, want_M)),
                  "counts": c.cnt.tolist()}))
dist.destroy_process_group()
"""


def test_share_ranges_over_gloo(tmp_path):
    script = tmp_path / "share_worker.py"
    script.write_text(SHARE_WORKER)
    port = _free_port()
    world = 3
    procs = []
    for r in range(world):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err
        o = json.loads(out.strip().splitlines()[-1])
        assert o["ok"] and o["counts"] == [3, 4, 5], o
