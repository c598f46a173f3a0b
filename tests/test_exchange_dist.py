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
