"""Incremental suffix synchronisation (streaming pack during source decoding, final synchronisation, assembly)
against the one-shot path: identical pages, identical merged table, logits within tolerance of the oracle."""
import numpy as np
import pytest

import synth
from tests.scenario import error_stats, oracle_reference

pytestmark = pytest.mark.gpu


def test_streamed_suffix_equals_one_shot_and_oracle():
    import torch
    import paper_2608_16477_b200 as kv
    from paper_2608_16477_b200 import streaming
    kv.load()
    s = synth.SHAPES["tiny-sharp"]
    bs, k, n = s.block_size, 128, 128 + 53
    ids = synth.token_ids(s, 4, n + 1)
    head = synth.head_weights(s, 4)
    model = kv.Model(s, head, lambda l: synth.layer_weights(s, 4, l))
    perm_s, perm_t = synth.block_permutation(5, 64), synth.block_permutation(6, 64)
    nb_total, nb_prefix = -(-n // bs), k // bs
    src, tgt = kv.PagedCache(s, 64, fill=0), kv.PagedCache(s, 64, fill=0)
    src_table = perm_s[:nb_total]
    tgt_prefix = perm_t[:nb_prefix]
    fresh = perm_t[nb_prefix:nb_prefix + 8]
    logits = torch.empty(s.vocab, dtype=torch.float32, device="cuda")
    # preparation trigger: split at k, epoch 3
    kv.kv_prefill_prefix(model, src, ids[:k], src_table[:nb_prefix])
    rx = streaming.SuffixReceiver(tgt, request_id=11, expected_epoch=3, k_split=k, max_suffix_blocks=8, fresh_block_ids=fresh)
    tx = streaming.SuffixStreamer(src, src_table, k, request_id=11, epoch=3, transport=streaming.LoopbackTransport(rx))
    # a message of a cancelled attempt is dropped on arrival
    assert not rx.on_block(streaming.BlockMessage(11, 2, nb_prefix, tx.slots[0]), tx.side)
    kv.kv_prefill_prefix(model, tgt, ids[:k], tgt_prefix)                      # target reconstructs the prefix
    sent_during_decode = 0
    for pos in range(k, n):                                                    # source keeps decoding
        kv.kv_decode_step(model, src, int(ids[pos]), pos, src_table[: pos // bs + 1], logits)
        tx.on_token(pos)
        if pos % 24 == 0:                                                      # the link gets a turn now and then
            sent_during_decode += tx.pump(max_blocks=1)
    backlog = tx.backlog_blocks
    residual = tx.final_sync(n)
    assert sent_during_decode + residual == nb_total - nb_prefix and residual == backlog + 1   # + boundary block
    assert sorted(tx.sent) == list(range(nb_prefix, nb_total)) and rx.dropped == 1
    merged = rx.assemble(tgt_prefix, n, epoch=3)
    assert np.array_equal(merged, np.concatenate([tgt_prefix, fresh[: nb_total - nb_prefix]]))
    torch.cuda.synchronize()
    # streamed pages == source pages (blocks never change once complete; the boundary block went last)
    for lb in range(nb_prefix, nb_total):
        assert torch.equal(src.pages([int(src_table[lb])]), tgt.pages([int(merged[lb])]))
    kv.kv_decode_step(model, tgt, int(ids[n]), n, list(merged), logits)      # resume at position n
    torch.cuda.synchronize()
    _, _, logits_ref = oracle_reference(s, 4, ids)
    st = error_stats(logits.cpu().numpy(), logits_ref)
    assert st["rel_l2"] <= 1e-2, st
    # a receiver that missed a block refuses to assemble ("without gaps")
    rx2 = streaming.SuffixReceiver(tgt, 11, 3, k, 8, perm_t[40:48])
    rx2.on_block(streaming.BlockMessage(11, 3, nb_prefix + 1, tx.slots[0]), tx.side)
    with pytest.raises(kv.KVError) as e:
        rx2.assemble(tgt_prefix, n, epoch=3)
    assert e.value.status in (-5, -6)
