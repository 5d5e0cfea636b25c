"""Incremental suffix synchronisation around the C-ABI operations (host-side orchestration only).

While the source keeps decoding, every suffix block that becomes complete is packed on a side stream into a
wire slot and handed to a transport together with its logical block index and the migration epoch; completed
blocks that have not been sent yet wait in a sender-side queue whose length at handover is the residual
transfer.  At handover the source sends the rest, including the partially filled boundary block.  The target
buffers what arrives (blocks of a stale epoch are dropped on arrival), and once the prefix has been
reconstructed and positions [k, n) are covered it assembles the merged block table with kv_unpack_assemble.
(Section 4.3, "Initialization and parallel preparation" and "Final synchronization and activation".)

Every byte is moved by kv_pack_blocks / kv_unpack_assemble; this module only sequences streams, events and
metadata.  `LoopbackTransport` delivers into a receiver on the same GPU (a device-to-device copy stands in for
the link).  `PeerTransport` is the two-process form: the sender issues one point-to-point send of a small
header and one of the wire slot per block (torch.distributed; NCCL over NVLink between two GPUs), and the
receiver posts the matching receive straight into its own receive buffer, so the payload lands in the target's
memory before any kernel of the target reads it.
"""
from __future__ import annotations

import contextlib
from collections import deque
from dataclasses import dataclass

import numpy as np

from . import binding as kv


@dataclass
class BlockMessage:
    request_id: int
    epoch: int
    logical_block: int
    wire: object          # device tensor holding one packed block (all layers, K and V)


class SuffixReceiver:
    """Target side: buffers arriving suffix blocks in a contiguous receive buffer and assembles the request."""

    def __init__(self, cache: kv.PagedCache, request_id: int, expected_epoch: int, k_split: int, max_suffix_blocks: int,
                 fresh_block_ids, device="cuda"):
        import torch
        self.cache, self.request_id, self.expected_epoch = cache, request_id, expected_epoch
        self.block_elems = cache.n_layers * 2 * (cache.page_bytes // 2)
        self.buffer = torch.empty(max_suffix_blocks * self.block_elems, dtype=torch.int16, device=device)
        self.fresh = [int(b) for b in fresh_block_ids]
        self.first_block = k_split // cache.block_size
        self.logical, self.dropped = [], 0

    def slot(self, i):
        return self.buffer[i * self.block_elems:(i + 1) * self.block_elems]

    def accepts(self, request_id: int, epoch: int) -> bool:
        """Whether an arriving block belongs to this migration attempt and still has a slot; a refused block
        counts as dropped."""
        ok = (epoch == self.expected_epoch and request_id == self.request_id
              and (len(self.logical) + 1) * self.block_elems <= self.buffer.numel())
        if not ok:
            self.dropped += 1
        return ok

    def next_slot(self):
        """The receive-buffer slot the next accepted block lands in."""
        return self.slot(len(self.logical))

    def commit(self, logical_block: int) -> None:
        """Records that the slot returned by next_slot() now holds `logical_block`."""
        self.logical.append(int(logical_block))

    def on_block(self, msg: BlockMessage, copy_stream) -> bool:
        """Stores one arriving block; returns False when it is discarded (stale epoch, foreign request, no room)."""
        import torch
        if not self.accepts(msg.request_id, msg.epoch):
            return False
        with torch.cuda.stream(copy_stream):
            self.next_slot().copy_(msg.wire, non_blocking=True)     # stands in for the link
        self.commit(msg.logical_block)
        return True

    def assemble(self, prefix_table, n_tokens_total: int, epoch: int, stream=None):
        """Unpacks the buffered blocks into fresh pages and returns the merged block table (raises KVError when
        [k, n) is not covered exactly once or the epoch is stale)."""
        n = len(self.logical)
        dst = self.fresh[:n]
        wire = self.buffer[: n * self.block_elems]
        return kv.kv_unpack_assemble(self.cache, wire, self.logical, dst, prefix_table, n_tokens_total, epoch=epoch,
                                     expected_epoch=self.expected_epoch, stream=stream)


class LoopbackTransport:
    def __init__(self, receiver: SuffixReceiver):
        self.receiver = receiver
        self.sent_blocks = 0

    def send(self, msg: BlockMessage, stream) -> None:
        self.receiver.on_block(msg, stream)
        self.sent_blocks += 1


def _on_stream(stream):
    import torch
    return torch.cuda.stream(stream) if stream is not None else contextlib.nullcontext()


class PeerTransport:
    """Point-to-point transport between the source's process and the target's (one process per GPU).

    Sender: `send(msg, stream)` enqueues, in stream order after the pack that filled the wire slot, a 4-word
    header (kind, request id, epoch, logical block) and the slot itself; `close(stream)` sends the end-of-stream
    header.  Receiver: `recv_into(receiver, stream)` takes one header, then receives the payload directly into
    the receiver's next buffer slot, or into a scratch slot when the receiver refuses the block (stale epoch,
    foreign request, buffer full), so that sends and receives always pair up.  Tensors live wherever the
    process group's backend expects them (device memory for NCCL, host memory for gloo); the transport moves
    bytes and metadata only.
    """

    KIND_BLOCK, KIND_END = 0, 1

    def __init__(self, peer: int, group=None):
        self.peer, self.group = int(peer), group
        self.sent_blocks = 0
        self._scratch = None

    def _header(self, like, kind, request_id=0, epoch=0, logical_block=0):
        import torch
        return torch.tensor([kind, request_id, epoch, logical_block], dtype=torch.int64, device=like.device)

    def send(self, msg: BlockMessage, stream=None) -> None:
        import torch.distributed as dist
        with _on_stream(stream):
            dist.send(self._header(msg.wire, self.KIND_BLOCK, msg.request_id, msg.epoch, msg.logical_block),
                      self.peer, group=self.group)
            dist.send(msg.wire, self.peer, group=self.group)
        self.sent_blocks += 1

    def close(self, like, stream=None) -> None:
        """Tells the receiver that no further block follows (`like`: any tensor on the sending device)."""
        import torch.distributed as dist
        with _on_stream(stream):
            dist.send(self._header(like, self.KIND_END), self.peer, group=self.group)

    def recv_into(self, receiver: SuffixReceiver, stream=None):
        """Receives one message.  Returns True (block stored), False (block dropped) or None (end of stream)."""
        import torch
        import torch.distributed as dist
        with _on_stream(stream):
            header = torch.empty(4, dtype=torch.int64, device=receiver.buffer.device)
            dist.recv(header, self.peer, group=self.group)
            kind, request_id, epoch, logical_block = (int(v) for v in header.tolist())   # waits for the header
            if kind == self.KIND_END:
                return None
            if receiver.accepts(request_id, epoch):
                dist.recv(receiver.next_slot(), self.peer, group=self.group)
                receiver.commit(logical_block)
                return True
            if self._scratch is None:
                self._scratch = torch.empty_like(receiver.slot(0))
            dist.recv(self._scratch, self.peer, group=self.group)
            return False


class SuffixStreamer:
    """Source side: turns completed suffix blocks into wire messages without stalling the decode stream."""

    def __init__(self, cache: kv.PagedCache, block_table, k_split: int, request_id: int, epoch: int, transport,
                 n_slots: int = 4, device="cuda"):
        import torch
        if k_split % cache.block_size:
            raise ValueError("the split position must be block-aligned")
        self.cache, self.table = cache, [int(b) for b in block_table]
        self.bs = cache.block_size
        self.request_id, self.epoch, self.transport = request_id, epoch, transport
        self.next_unqueued = k_split // self.bs          # first logical block not yet queued
        self.queue = deque()                              # completed, not yet sent (sender-side queue)
        self.side = torch.cuda.Stream(device=device)
        block_elems = cache.n_layers * 2 * (cache.page_bytes // 2)
        self.slots = [torch.empty(block_elems, dtype=torch.int16, device=device) for _ in range(n_slots)]
        self.slot_free = [None] * n_slots                 # event after which the slot may be overwritten
        self.cursor = 0
        self.sent = []

    @property
    def backlog_blocks(self) -> int:
        return len(self.queue)

    def on_token(self, pos: int, decode_stream=None) -> None:
        """Call after the decode step that wrote K/V of position `pos` has been enqueued."""
        import torch
        if (pos + 1) % self.bs == 0:
            ev = torch.cuda.Event()
            ev.record(decode_stream or torch.cuda.current_stream())
            self.queue.append((self.next_unqueued, ev))
            self.next_unqueued += 1

    def _send(self, logical_block: int, ready_event) -> None:
        import torch
        i = self.cursor % len(self.slots)
        self.cursor += 1
        if ready_event is not None:
            self.side.wait_event(ready_event)
        if self.slot_free[i] is not None:
            self.side.wait_event(self.slot_free[i])
        kv.kv_pack_blocks(self.cache, [self.table[logical_block]], self.slots[i], stream=self.side)
        self.transport.send(BlockMessage(self.request_id, self.epoch, logical_block, self.slots[i]), self.side)
        done = torch.cuda.Event()
        done.record(self.side)
        self.slot_free[i] = done
        self.sent.append(logical_block)

    def pump(self, max_blocks: int | None = None) -> int:
        """Packs and sends queued blocks on the side stream; returns how many were sent."""
        n = 0
        while self.queue and (max_blocks is None or n < max_blocks):
            logical_block, ev = self.queue.popleft()
            self._send(logical_block, ev)
            n += 1
        return n

    def final_sync(self, n_tokens_total: int, decode_stream=None) -> int:
        """Handover: sends every unsent completed block and the partially filled boundary block; returns the
        number of blocks that were still outstanding (the residual transfer)."""
        import torch
        ev = torch.cuda.Event()
        ev.record(decode_stream or torch.cuda.current_stream())
        residual = self.pump()
        last_block = -(-n_tokens_total // self.bs)
        while self.next_unqueued < last_block:            # the boundary block (n % Bs valid slots)
            self._send(self.next_unqueued, ev)
            self.next_unqueued += 1
            residual += 1
        (decode_stream or torch.cuda.current_stream()).wait_stream(self.side)
        return residual
