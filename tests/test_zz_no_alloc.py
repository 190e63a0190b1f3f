"""The allocation-free prune entry point gives the same bits as the context-based one.

Collected last on purpose (file name): a run that stops at the first failure has then
already run every other test.  The check is done twice in a row with different sizes,
because the entry point's scratch is one fixed array inside the library that still holds
the previous call's contents; the second, smaller call must not be disturbed by them.
"""
import numpy as np
import pytest
import torch

from paper_2601_07891_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu


def _one_round(binding, ctx, oracle, seq_lens, tau, w, seed, D=128, H=8):
    T = int(sum(seq_lens))
    B = len(seq_lens)
    g = torch.Generator().manual_seed(seed)
    scores = torch.randn(T, H, generator=g).cuda()
    K, V = synth.keys_values(H, T, D, seed)
    K, V = K.cuda(), V.cuda()
    cu = torch.from_numpy(synth.cu_seqlens(seq_lens)).cuda() if B > 1 else None
    poison = lambda: parity.poison_like(K)
    # existing entry point (context scratch from cudaMalloc)
    K_ref, V_ref = poison(), poison()
    len_ref = torch.full((B, H), -1, dtype=torch.int32, device="cuda")
    ctx.prune_prefill(K, V, scores, tau, w, cu_seqlens=cu, K_out=K_ref, V_out=V_ref, lengths=len_ref)
    # new entry point (static scratch), straight through the C ABI
    K_new, V_new = poison(), poison()
    len_new = torch.full((B, H), -1, dtype=torch.int32, device="cuda")
    binding.kvzap_prune_prefill_noalloc(K, V, scores, cu, B, tau, w, K_new, V_new, len_new)
    torch.cuda.synchronize()
    assert torch.equal(len_new, len_ref)
    assert int(len_ref.sum()) > 0
    assert torch.equal(K_new.view(torch.int16), K_ref.view(torch.int16))      # bit-exact, poison rows included
    assert torch.equal(V_new.view(torch.int16), V_ref.view(torch.int16))
    # and against the oracle's mask + ordered gather of the same scores (rows past the lengths keep their poison)
    cu_np = synth.cu_seqlens(seq_lens) if B > 1 else None
    parity.check_compaction(oracle, K.cpu(), V.cpu(), scores.cpu().numpy(), tau, w, cu_np, K_new.cpu(), V_new.cpu(), len_new)


def test_noalloc_matches_context_entry_point_two_calls_in_a_row(oracle):
    from paper_2601_07891_b200 import binding
    binding.load()
    ctx = binding.Kvzap(256, 0, 8, 128, 1, max_tokens=8192, max_seqs=8)
    _one_round(binding, ctx, oracle, [5000, 1, 0, 2999], 0.43, 128, seed=1)      # 8000 tokens, several blocks, ragged
    _one_round(binding, ctx, oracle, [333], -0.2, 16, seed=2)                    # smaller: stale scratch must not matter
    ctx.close()
    ctx = binding.Kvzap(256, 0, 3, 64, 1, max_tokens=2048, max_seqs=2)   # other shape parameters
    _one_round(binding, ctx, oracle, [700, 700], 0.9, 0, seed=3, D=64, H=3)
    ctx.close()


def test_noalloc_rejects_sizes_beyond_the_static_scratch():
    from paper_2601_07891_b200 import binding
    H, D = 8, 8
    T = binding.NOALLOC_MAX_TOKENS + 1
    K = torch.zeros(H, T, D, dtype=torch.bfloat16, device="cuda")
    scores = torch.zeros(T, H, device="cuda")
    lengths = torch.zeros(1, H, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.KvzapError) as ei:
        binding.kvzap_prune_prefill_noalloc(K, K, scores, None, 1, 0.0, 0, K.clone(), K.clone(), lengths)
    assert ei.value.status == 2 and "KVZAP_NOALLOC_MAX_TOKENS" in str(ei.value)
    cu = torch.zeros(binding.NOALLOC_MAX_SEQS + 2, dtype=torch.int32, device="cuda")
    small = torch.zeros(H, 16, D, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.KvzapError) as ei:
        binding.kvzap_prune_prefill_noalloc(small, small, torch.zeros(16, H, device="cuda"), cu,
                                            binding.NOALLOC_MAX_SEQS + 1, 0.0, 0, small.clone(), small.clone(), lengths)
    assert ei.value.status == 2 and "KVZAP_NOALLOC_MAX_SEQS" in str(ei.value)
