"""The exchange between tensor-parallel ranks (Section 5: an all-gather of the payloads, then a local reduction).

One process per GPU.  Rank r owns shard r: it calibrates and quantises only its own partial sums, and every
rank dequantises and sums all N payloads.  Three pieces:

* `share_ranges`       the static ranges are per (device, feature); the top-k set needs their sum over the
                       devices, so the ranks all-gather their (m, M, count) rows once after calibration and
                       every rank builds identical tables.
* `AllGatherExchange`  the payload bytes through the collective library (`all_gather_into_tensor`): the
                       baseline, and the form that also runs on CPU tensors (gloo).
* `PushExchange`       the fused form: the quantiser stores its payload straight into its slot of every
                       rank's receive buffer (peer-mapped symmetric memory, plain stores over NVLink), then
                       publishes an arrival word; the reducing side waits for its N words with a limit and
                       reads local memory only.  No collective call in the step.

Only argument marshalling and buffer bookkeeping happen here; the arithmetic is in the CUDA library."""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

try:  # torch.distributed is optional at import time (single-process use needs none of it)
    import torch.distributed as dist
except Exception:  # pragma: no cover
    dist = None


def _world(group=None):
    if dist is None or not dist.is_available() or not dist.is_initialized():
        return 0, 1
    return dist.get_rank(group), dist.get_world_size(group)


@dataclass(frozen=True)
class ReceiveLayout:
    """Byte layout of one rank's receive buffer: 2 slot sets x N payload slots, then 2 x N arrival words.

    Two sets alternate with the step number.  Every step waits for all N arrivals, so a rank that has
    finished step e knows that every rank has pushed step e, hence finished reading step e-1: the set of
    step e+1 (the one of step e-1) is free to be overwritten."""
    n_ranks: int
    payload_bytes: int

    @property
    def slot_bytes(self) -> int:
        return (self.payload_bytes + 255) // 256 * 256

    @property
    def words_offset(self) -> int:
        return 2 * self.n_ranks * self.slot_bytes

    @property
    def total_bytes(self) -> int:
        return self.words_offset + (2 * self.n_ranks * 4 + 255) // 256 * 256

    def slot(self, step: int, src_rank: int) -> int:
        """Byte offset of the slot that src_rank's payload of this step lands in."""
        assert 0 <= src_rank < self.n_ranks
        return ((step & 1) * self.n_ranks + src_rank) * self.slot_bytes

    def word(self, step: int, src_rank: int) -> int:
        """Byte offset of the arrival word beside that slot."""
        assert 0 <= src_rank < self.n_ranks
        return self.words_offset + 4 * ((step & 1) * self.n_ranks + src_rank)

    @staticmethod
    def epoch(step: int) -> int:
        """The tag of a step: never 0 (a fresh buffer is zero-filled), distinct for the two steps that
        share a slot set in any window of 2^31 steps."""
        return (step % 0x7FFFFFFF) + 1


def gather_rows(row: np.ndarray, group=None) -> np.ndarray:
    """All-gather one equally shaped numpy row per rank -> [world, ...] in rank order (any backend)."""
    rank, world = _world(group)
    if world == 1:
        return row[None].copy()
    dev = "cuda" if dist.get_backend(group) == "nccl" else "cpu"
    mine = torch.from_numpy(np.ascontiguousarray(row)).to(dev)
    out = torch.empty((world,) + tuple(mine.shape), dtype=mine.dtype, device=dev)
    dist.all_gather_into_tensor(out, mine[None].contiguous(), group=group)
    return out.cpu().numpy()


def share_ranges(tpq, count: int, group=None) -> None:
    """After rank r has folded `count` calibration sequences into shard r of its context: give every rank
    all N rows of the moving-average state (Eq. 1-2), so that every rank derives the same feature set."""
    rank, world = _world(group)
    if world != tpq.N:
        raise ValueError(f"context has {tpq.N} shards, the group {world} ranks")
    m, M = tpq.get_ranges(with_R=False)
    rows = gather_rows(np.concatenate([m[rank], M[rank]]).astype(np.float32), group)
    cnt = gather_rows(np.asarray([count], dtype=np.int64), group).reshape(world)
    E = tpq.E
    tpq.set_ranges(np.ascontiguousarray(rows[:, :E]), np.ascontiguousarray(rows[:, E:]), cnt)


class AllGatherExchange:
    """Payload bytes through the collective library.  `gather` works on CUDA tensors (nccl) and on CPU
    tensors (gloo); the result is [N, payload_bytes] in rank order."""

    def __init__(self, payload_bytes: int, group=None, device=None):
        self.group = group
        self.rank, self.world = _world(group)
        self.payload_bytes = payload_bytes
        self.device = device
        self._out = None

    def gather(self, payload: torch.Tensor) -> torch.Tensor:
        assert payload.dtype == torch.uint8 and payload.numel() == self.payload_bytes
        if self._out is None or self._out.device != payload.device:
            self._out = torch.empty((self.world, self.payload_bytes), dtype=torch.uint8, device=payload.device)
        if self.world == 1:
            self._out[0].copy_(payload)
        else:
            dist.all_gather_into_tensor(self._out, payload.reshape(1, -1), group=self.group)
        return self._out

    def step(self, tpq, y_ptr: int, T: int, out_ptr: int, out_dtype: int, payload: torch.Tensor, stream: int = 0,
             bias_ptr: int | None = None) -> None:
        """quantize_pack(own shard) -> all-gather -> dequant_reduce, on the current CUDA stream."""
        tpq.quantize_pack(self.rank, y_ptr, T, payload.data_ptr(), payload.numel(), stream=stream)
        allp = self.gather(payload)
        tpq.dequant_reduce([allp[i].data_ptr() for i in range(self.world)], T, out_ptr, out_dtype, stream=stream,
                           bias_ptr=bias_ptr)


@dataclass
class PeerBuffers:
    """One receive buffer per rank, each mapped by every rank: peer_ptrs[p] is the address at which THIS rank
    reaches rank p's buffer (peer_ptrs[rank] is its own).  `keep` holds whatever owns the memory."""
    rank: int
    peer_ptrs: list
    keep: object = None


def open_peer_buffers(total_bytes: int, group=None, device=None) -> PeerBuffers:
    """Allocate this rank's receive buffer, zero it and exchange the mappings: symmetric memory when there is
    more than one rank (every rank maps every peer's buffer), a plain device tensor otherwise."""
    rank, world = _world(group)
    device = device if device is not None else torch.device("cuda", torch.cuda.current_device())
    if world == 1:
        buf = torch.zeros(total_bytes, dtype=torch.uint8, device=device)
        return PeerBuffers(0, [buf.data_ptr()], buf)
    import torch.distributed._symmetric_memory as symm_mem
    buf = symm_mem.empty(total_bytes, dtype=torch.uint8, device=device)
    buf.zero_()
    g = group if group is not None else dist.group.WORLD
    hdl = symm_mem.rendezvous(buf, g)
    ptrs = [int(p) for p in hdl.buffer_ptrs]
    torch.cuda.synchronize(device)
    dist.barrier(group=group)  # every buffer is zeroed before anyone pushes
    return PeerBuffers(rank, ptrs, (buf, hdl))


class PushExchange:
    """The fused exchange.  Per step s, rank r stores its payload into slot (s & 1, r) of EVERY rank's receive
    buffer and then the step's tag into the arrival word beside each copy; the reduction on rank r waits for
    the N words of set s & 1 in its OWN buffer and reads its own N slots.  Peers are only ever stored to.

    `buffers` (a PeerBuffers) may be handed in by the caller, e.g. addresses obtained from another
    allocator, or host-made integers in a test of this bookkeeping; by default open_peer_buffers is used."""

    def __init__(self, tpq, T: int, group=None, device=None, timeout_ns: int = 1_000_000_000, buffers=None,
                 world: int | None = None):
        self.tpq = tpq
        self.T = T
        self.group = group
        self.rank, self.world = _world(group)
        if buffers is not None:
            self.rank = buffers.rank
            self.world = world if world is not None else len(buffers.peer_ptrs)
        if self.world != tpq.N:
            raise ValueError(f"context has {tpq.N} shards, the group {self.world} ranks")
        self.layout = ReceiveLayout(self.world, tpq.payload_bytes(T))
        self.timeout_ns = timeout_ns
        self.step_no = 0
        self.buffers = buffers if buffers is not None else open_peer_buffers(self.layout.total_bytes, group, device)
        if len(self.buffers.peer_ptrs) != self.world:
            raise ValueError(f"{len(self.buffers.peer_ptrs)} peer mappings for {self.world} ranks")
        self.peer_ptrs = list(self.buffers.peer_ptrs)

    def push_args(self, step: int):
        """(destinations, arrival words, tag) of this rank's push in `step`: one pair per rank, in rank order."""
        L, r = self.layout, self.rank
        return ([p + L.slot(step, r) for p in self.peer_ptrs], [p + L.word(step, r) for p in self.peer_ptrs],
                L.epoch(step))

    def reduce_args(self, step: int):
        """(payload addresses in device order, first arrival word, tag) of this rank's reduction in `step`:
        all in its own buffer; the N words of a set are adjacent, one wait covers them."""
        L, mine = self.layout, self.peer_ptrs[self.rank]
        return [mine + L.slot(step, i) for i in range(self.world)], mine + L.word(step, 0), L.epoch(step)

    def step(self, y_ptr: int, out_ptr: int, out_dtype: int, stream: int = 0, bias_ptr: int | None = None) -> None:
        """One synchronisation: push own shard to every rank, wait for all N arrivals, reduce locally."""
        s = self.step_no
        dst, words, epoch = self.push_args(s)
        self.tpq.quantize_pack_push(self.rank, y_ptr, self.T, dst, words, self.layout.slot_bytes, epoch, stream=stream)
        payloads, first_word, epoch = self.reduce_args(s)
        self.tpq.dequant_reduce(payloads, self.T, out_ptr, out_dtype, stream=stream, bias_ptr=bias_ptr,
                                arrived_ptr=first_word, epoch=epoch, timeout_ns=self.timeout_ns)
        self.step_no += 1
