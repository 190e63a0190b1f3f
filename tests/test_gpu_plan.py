"""kvzap_prefill_plan (the write plan: where every kept (token, head) pair belongs, no K/V byte moved)
against the oracle: slots, lengths and page tables bit for bit given the GPU's scores, and the property
that matters to a caller -- a producer that writes each kept row to its slot ends up with exactly the
ordered compaction."""
import numpy as np
import pytest
import torch

from paper_2601_07891_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_2601_07891_b200 import binding as b
    b.load()
    return b


def _weights(d_model, hidden, H, seed):
    return synth.mlp_weights(d_model, hidden, H, seed, "cpu", 0.3) if hidden else synth.linear_weights(d_model, H, seed, "cpu", 0.3)


@pytest.mark.parametrize("seq_lens,hidden,H,P", [([1000], 0, 8, 0), ([300, 0, 77, 1500, 1], 128, 8, 0), ([4097], 64, 5, 0),
                                                 ([1000], 0, 8, 16), ([300, 0, 77, 1500, 1], 128, 8, 7), ([20000, 13000], 0, 8, 16)])
def test_plan_matches_oracle_and_scatter_gives_the_compaction(binding, oracle, seq_lens, hidden, H, P):
    d_model, D, tau, w = 256, 64, 0.2, 32
    T, B = int(sum(seq_lens)), len(seq_lens)
    ctx = binding.Kvzap(d_model, hidden, H, D, 1, T, max_seqs=B)
    wts = _weights(d_model, hidden, H, 11 + hidden)
    ctx.set_weights(0, *[parity.dev(x) for x in wts])
    X = synth.hidden_states(T, d_model, seed=21)
    K, V = synth.keys_values(H, T, D, seed=22)
    cu = synth.cu_seqlens(seq_lens)
    cu_dev = torch.from_numpy(cu).cuda() if B > 1 else None
    cu_arg = cu if B > 1 else None
    slot = torch.full((T, H), -9, dtype=torch.int32, device="cuda")
    lengths = torch.full((B, H), -1, dtype=torch.int32, device="cuda")
    scores = torch.empty(T, H, dtype=torch.float32, device="cuda")
    if P:
        n_pool, max_pages, first = H * (T // P + B + 1) + 3, max(seq_lens) // P + 2, 2
        table = torch.full((B * H, max_pages), -1, dtype=torch.int32, device="cuda")
        used = torch.zeros(1, dtype=torch.int32, device="cuda")
        binding.kvzap_prefill_plan(ctx.handle, 0, parity.dev(X), cu_dev, B, tau, w, slot, lengths, scores, page_tokens=P,
                                   n_pages_pool=n_pool, first_page=first, page_table=table, n_pages_used=used)
    else:
        binding.kvzap_prefill_plan(ctx.handle, 0, parity.dev(X), cu_dev, B, tau, w, slot, lengths, scores)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    want, _ = parity.check_scores(oracle, scores, X, wts)
    s = scores.cpu().numpy()
    keep = parity.check_mask_band(oracle, s, want, tau, w, cu_arg)
    got_slot = slot.cpu().numpy()
    Kb, Vb = synth.bits(K), synth.bits(V)
    if P:
        ref_slot, ref_len, ref_tab, ref_used = oracle.plan(keep, cu_arg, page_tokens=P, n_pages_pool=n_pool,
                                                           max_pages_per_list=max_pages, first_page=first)
        np.testing.assert_array_equal(table.cpu().numpy(), ref_tab)
        assert int(used.item()) == ref_used
    else:
        ref_slot, ref_len = oracle.plan(keep, cu_arg)
    np.testing.assert_array_equal(got_slot, ref_slot)
    np.testing.assert_array_equal(lengths.cpu().numpy(), ref_len)
    # the producer's side: every kept row straight to its slot (a scatter written with torch indexing here)
    t_idx, h_idx = np.nonzero(got_slot >= 0)
    rows = got_slot[t_idx, h_idx].astype(np.int64)
    if P:
        Kp = np.full((n_pool * P, D), parity.POISON, dtype=np.uint16)
        Vp = np.full((n_pool * P, D), parity.POISON, dtype=np.uint16)
        Kp[rows], Vp[rows] = Kb[h_idx, t_idx], Vb[h_idx, t_idx]
        Kr, Vr, _tab, _ln, _n = oracle.compact_paged(Kb, Vb, keep, P, n_pool, max_pages, cu_seqlens=cu_arg, first_page=first,
                                                     fill=parity.POISON)
        np.testing.assert_array_equal(Kp.reshape(n_pool, P, D), Kr)
        np.testing.assert_array_equal(Vp.reshape(n_pool, P, D), Vr)
    else:
        seq_of = np.searchsorted(cu, t_idx, side="right") - 1
        Ko = np.full_like(Kb, parity.POISON)
        Vo = np.full_like(Vb, parity.POISON)
        Ko[h_idx, cu[seq_of] + rows], Vo[h_idx, cu[seq_of] + rows] = Kb[h_idx, t_idx], Vb[h_idx, t_idx]
        Kr, Vr, _ln = oracle.compact(Kb, Vb, keep, cu_arg, fill=parity.POISON)
        np.testing.assert_array_equal(Ko, Kr)
        np.testing.assert_array_equal(Vo, Vr)
    ctx.close()


def test_plan_without_scores_buffer_and_pool_too_small(binding, oracle):
    d_model, H, D, T, P = 256, 8, 64, 600, 16
    ctx = binding.Kvzap(d_model, 0, H, D, 1, T)
    wts = _weights(d_model, 0, H, 3)
    ctx.set_weights(0, *[parity.dev(x) for x in wts])
    X = parity.dev(synth.hidden_states(T, d_model, seed=5))
    slot = torch.full((T, H), -9, dtype=torch.int32, device="cuda")
    lengths = torch.zeros(1, H, dtype=torch.int32, device="cuda")
    binding.kvzap_prefill_plan(ctx.handle, 0, X, None, 1, 0.1, 16, slot, lengths)          # scores kept inside the context
    torch.cuda.synchronize()
    s = ctx.score(0, X).cpu().numpy()
    ref_slot, ref_len = oracle.plan(oracle.keep_mask(s, 0.1, 16))
    np.testing.assert_array_equal(slot.cpu().numpy(), ref_slot)
    np.testing.assert_array_equal(lengths.cpu().numpy(), ref_len)
    table = torch.full((H, 40), -1, dtype=torch.int32, device="cuda")
    used = torch.full((1,), 5, dtype=torch.int32, device="cuda")
    binding.kvzap_prefill_plan(ctx.handle, 0, X, None, 1, 0.1, 16, slot, lengths, None, page_tokens=P, n_pages_pool=10,
                               first_page=0, page_table=table, n_pages_used=used)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 4 and int(used.item()) == 0 and (slot == -1).all()
    np.testing.assert_array_equal(lengths.cpu().numpy(), ref_len)
    ctx.close()
