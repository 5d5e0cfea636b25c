"""The decode-attention entry point for callers that cannot allocate device memory.

Hosts such as a serving engine whose start-up pools own all of HBM, or the activation path right after a
handover, have no scratch buffer to give and must not call cudaMalloc.  kv_op_paged_attention_noalloc keeps
its split-KV partials in a fixed array inside the library instead.  This test calls it through the C ABI
twice in a row (different queries, layers and context lengths, so the second call runs over what the first
left in the shared array) and checks each result against kv_op_paged_attention, which takes its scratch from
the caller.  It lives in its own file, collected last, and also passes when run alone in a fresh process.
"""
import numpy as np
import pytest

import synth

pytestmark = pytest.mark.gpu


def test_noalloc_matches_scratch_variant_twice():
    import torch
    import paper_2608_16477_b200 as kv
    kv.load()
    s = synth.ModelShape("pa", n_layers=2, hidden=64, n_q_heads=8, n_kv_heads=2, head_dim=128, ffn=64, vocab=16)
    nb = 128
    cache = kv.PagedCache(s, nb)
    g = torch.Generator(device="cuda").manual_seed(5)
    vals = torch.randn(cache.data.shape, generator=g, device="cuda").to(torch.bfloat16)
    cache.data.copy_(vals.view(torch.int16))
    table = torch.from_numpy(synth.block_permutation(11, nb)).cuda()
    for call, (n_ctx, layer) in enumerate([(1500, 1), (333, 0)]):
        q = torch.randn(8, 128, generator=g, device="cuda")
        want = torch.empty(8, 128, dtype=torch.float32, device="cuda")
        scratch = torch.empty(kv.kv_paged_attention_scratch_bytes(8, 128, n_ctx), dtype=torch.uint8, device="cuda")
        kv.kv_op_paged_attention(q, cache, layer, table, n_ctx, scratch, want)
        got = torch.full((8, 128), float("nan"), dtype=torch.float32, device="cuda")
        kv.kv_op_paged_attention_noalloc(q, cache, layer, table, n_ctx, got)
        torch.cuda.synchronize()
        assert torch.isfinite(got).all(), f"call {call}"
        assert torch.max(torch.abs(got - want)).item() < 1e-4, f"call {call}"


def test_noalloc_rejects_contexts_beyond_its_array():
    import torch
    import paper_2608_16477_b200 as kv
    kv.load()
    s = synth.ModelShape("pa", n_layers=1, hidden=64, n_q_heads=64, n_kv_heads=8, head_dim=128, ffn=64, vocab=16)
    cache = kv.PagedCache(s, 8)
    q = torch.zeros(64, 128, device="cuda")
    out = torch.zeros(64, 128, device="cuda")
    table = torch.zeros(8, dtype=torch.int32, device="cuda")
    too_long = 16128 + 1              # one 128-key split beyond what 4 MiB of partials can hold for 64 heads of 128
    assert kv.kv_paged_attention_scratch_bytes(64, 128, 16128) <= 4 * 1024 * 1024
    assert kv.kv_paged_attention_scratch_bytes(64, 128, too_long) > 4 * 1024 * 1024
    with pytest.raises(kv.KVError) as e:
        kv.kv_op_paged_attention_noalloc(q, cache, 0, table, too_long, out)
    assert e.value.status == -10      # KV_ERR_WORKSPACE: nothing was launched
