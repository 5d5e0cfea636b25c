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
the link); a two-GPU transport would replace that copy by a send/receive of the same wire slot into the
receiver's own memory.
"""
from __future__ import annotations

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

    def on_block(self, msg: BlockMessage, copy_stream) -> bool:
        """Stores one arriving block; returns False when it is discarded (stale epoch, foreign request, no room)."""
        import torch
        if msg.epoch != self.expected_epoch or msg.request_id != self.request_id:
            self.dropped += 1
            return False
        if len(self.logical) * self.block_elems >= self.buffer.numel():
            self.dropped += 1
            return False
        with torch.cuda.stream(copy_stream):
            self.slot(len(self.logical)).copy_(msg.wire, non_blocking=True)     # stands in for the link
        self.logical.append(int(msg.logical_block))
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
