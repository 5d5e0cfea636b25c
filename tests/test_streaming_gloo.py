"""The one exchange step of the path (source packs, the wire slot crosses the link, the target buffers it in its
own memory) between two processes on CPU: two gloo ranks drive PeerTransport and SuffixReceiver with wire blocks
of seeded pattern bytes.  Checks: every accepted block lands in the receiver's buffer byte for byte and in arrival
order, logical indices follow the headers, blocks of a stale epoch or a foreign request are dropped without
breaking the send/receive pairing, a full buffer refuses further blocks, and the end-of-stream header ends the
loop.  (Section 4.3: incremental suffix synchronisation, final synchronisation, epoch check on arrival.)"""
import os
import socket
from types import SimpleNamespace

import numpy as np
import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist  # noqa: E402
import torch.multiprocessing as mp  # noqa: E402

import synth  # noqa: E402
from paper_2608_16477_b200 import streaming  # noqa: E402

GEOM = SimpleNamespace(n_layers=3, page_bytes=16 * 2 * 8 * 2, block_size=16)     # 3 layers, pages of 512 bytes
BLOCK_BYTES = GEOM.n_layers * 2 * GEOM.page_bytes
K_SPLIT, EPOCH, REQUEST = 32, 7, 41
# (request id, epoch, logical block): two good blocks, a stale epoch, a foreign request, a good block out of
# order, and one more than the receive buffer (4 slots) can hold
MESSAGES = [(REQUEST, EPOCH, 2), (REQUEST, EPOCH, 3), (REQUEST, EPOCH - 1, 4), (REQUEST + 1, EPOCH, 4),
            (REQUEST, EPOCH, 5), (REQUEST, EPOCH, 4), (REQUEST, EPOCH, 6)]


def _wire(i):
    raw = synth.pattern_bytes(1000 + i, 0, BLOCK_BYTES)
    return torch.from_numpy(np.frombuffer(raw, dtype=np.int16).copy())


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE="2")
    dist.init_process_group("gloo", rank=rank, world_size=2)
    try:
        link = streaming.PeerTransport(peer=1 - rank)
        if rank == 0:                                            # the source
            for i, (req, epoch, logical) in enumerate(MESSAGES):
                link.send(streaming.BlockMessage(req, epoch, logical, _wire(i)))
            link.close(_wire(0))
            out.put((0, link.sent_blocks, None, None, None))
        else:                                                    # the target
            rx = streaming.SuffixReceiver(GEOM, REQUEST, EPOCH, K_SPLIT, max_suffix_blocks=4,
                                          fresh_block_ids=[9, 8, 7, 6], device="cpu")
            verdicts = []
            while True:
                v = link.recv_into(rx)
                if v is None:
                    break
                verdicts.append(v)
            out.put((1, verdicts, list(rx.logical), rx.dropped, rx.buffer.numpy().tobytes()))
    finally:
        dist.destroy_process_group()


def test_blocks_cross_the_link_into_the_receivers_buffer():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    results = dict((r[0], r[1:]) for r in (q.get(timeout=120) for _ in range(2)))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert results[0][0] == len(MESSAGES)
    verdicts, logical, dropped, buf = results[1]
    assert verdicts == [True, True, False, False, True, True, False]
    assert logical == [2, 3, 5, 4]                              # arrival order, as the headers said
    assert dropped == 3
    accepted = [0, 1, 4, 5]
    expect = b"".join(synth.pattern_bytes(1000 + i, 0, BLOCK_BYTES) for i in accepted)
    assert buf == expect
