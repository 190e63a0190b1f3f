"""The host-buffer entry points (inputs and outputs in host memory, copies inside the call) against
the oracle: several layers in one pipelined call, dense-ragged and paged, pinned and pageable memory,
and the one-layer calls built on it."""
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


def _maybe_pin(t, pin):
    return t.pin_memory() if pin else t


@pytest.mark.parametrize("seq_lens,hidden,pin", [([3000], 128, True), ([700, 0, 1300, 77], 0, True), ([1500, 200], 128, False)])
def test_layers_host_dense_matches_oracle(binding, oracle, seq_lens, hidden, pin):
    d_model, H, D, L, tau, w = 256, 8, 64, 3, 0.2, 32
    T, B = int(sum(seq_lens)), len(seq_lens)
    ctx = binding.Kvzap(d_model, hidden, H, D, L, T, max_seqs=B)
    weights = []
    for l in range(L):
        wts = synth.mlp_weights(d_model, hidden, H, 30 + l, "cpu", 0.3) if hidden else synth.linear_weights(d_model, H, 30 + l, "cpu", 0.3)
        weights.append(wts)
        ctx.set_weights(l, *[parity.dev(x) for x in wts])
    cu = synth.cu_seqlens(seq_lens)
    cu_t = torch.from_numpy(cu) if B > 1 else None
    cu_arg = cu if B > 1 else None
    Xs = [_maybe_pin(synth.hidden_states(T, d_model, 100 + l), pin) for l in range(L)]
    KVs = [synth.keys_values(H, T, D, 200 + l) for l in range(L)]
    Ks, Vs = [_maybe_pin(kv[0], pin) for kv in KVs], [_maybe_pin(kv[1], pin) for kv in KVs]
    Kos = [_maybe_pin(parity.poison_like(Ks[l]), pin) for l in range(L)]
    Vos = [_maybe_pin(parity.poison_like(Ks[l]), pin) for l in range(L)]
    lens = [_maybe_pin(torch.full((B, H), -1, dtype=torch.int32), pin) for _ in range(L)]
    scs = [_maybe_pin(torch.empty(T, H, dtype=torch.float32), pin) if l != 1 else None for l in range(L)]
    binding.kvzap_prefill_layers_host(ctx.handle, 0, Xs, Ks, Vs, cu_t, B, tau, w, Kos, Vos, lens, scs)
    assert ctx.poll_status() == 0
    for l in range(L):
        want = oracle.score(synth.bits(Xs[l]), parity.weights_to_oracle(weights[l]))
        if scs[l] is not None:
            s = scs[l].numpy()
            assert np.abs(s - want).max() <= parity.SCORE_ATOL
        else:                                           # scores not asked for: take them from the device call
            s = ctx.score(l, parity.dev(Xs[l])).cpu().numpy()
        parity.check_mask_band(oracle, s, want, tau, w, cu_arg)
        parity.check_compaction(oracle, Ks[l], Vs[l], s, tau, w, cu_arg, Kos[l], Vos[l], lens[l])
    # the one-layer call gives the same bits
    Ko1, Vo1 = parity.poison_like(Ks[2]), parity.poison_like(Ks[2])
    len1 = torch.full((B, H), -1, dtype=torch.int32)
    binding.kvzap_prefill_fused_host(ctx.handle, 2, Xs[2], Ks[2], Vs[2], cu_t, B, tau, w, Ko1, Vo1, len1, None)
    assert torch.equal(len1, lens[2])
    assert torch.equal(Ko1.view(torch.int16), Kos[2].view(torch.int16)) and torch.equal(Vo1.view(torch.int16), Vos[2].view(torch.int16))
    ctx.close()


@pytest.mark.parametrize("seq_lens,P", [([2500], 16), ([600, 900, 0, 31], 5)])
def test_layers_host_paged_matches_oracle(binding, oracle, seq_lens, P):
    d_model, hidden, H, D, L, tau, w = 256, 64, 8, 64, 3, 0.25, 16
    T, B = int(sum(seq_lens)), len(seq_lens)
    ctx = binding.Kvzap(d_model, hidden, H, D, L, T, max_seqs=B)
    weights = []
    for l in range(L):
        wts = synth.mlp_weights(d_model, hidden, H, 60 + l, "cpu", 0.3)
        weights.append(wts)
        ctx.set_weights(l, *[parity.dev(x) for x in wts])
    cu = synth.cu_seqlens(seq_lens)
    cu_t = torch.from_numpy(cu) if B > 1 else None
    cu_arg = cu if B > 1 else None
    n_pool, max_pages = H * (T // P + B + 1) + 9, max(seq_lens) // P + 2
    first = [0, 4, 7]
    Xs = [synth.hidden_states(T, d_model, 300 + l).pin_memory() for l in range(L)]
    KVs = [synth.keys_values(H, T, D, 400 + l) for l in range(L)]
    Ks, Vs = [kv[0].pin_memory() for kv in KVs], [kv[1].pin_memory() for kv in KVs]
    pools_k = [torch.full((n_pool, P, D), -5.0, dtype=torch.bfloat16).pin_memory() for _ in range(L)]
    pools_v = [torch.full((n_pool, P, D), -5.0, dtype=torch.bfloat16).pin_memory() for _ in range(L)]
    tabs = [torch.full((B * H, max_pages), -1, dtype=torch.int32).pin_memory() for _ in range(L)]
    lens = [torch.zeros(B, H, dtype=torch.int32).pin_memory() for _ in range(L)]
    used = [torch.zeros(1, dtype=torch.int32).pin_memory() for _ in range(L)]
    scs = [torch.empty(T, H, dtype=torch.float32).pin_memory() for _ in range(L)]
    binding.kvzap_prefill_layers_host(ctx.handle, 0, Xs, Ks, Vs, cu_t, B, tau, w, pools_k, pools_v, lens, scs,
                                      page_tokens=P, first_page=first, page_table=tabs, n_pages_used=used)
    assert ctx.poll_status() == 0
    fill = int(synth.bits(torch.tensor([-5.0], dtype=torch.bfloat16))[0])
    for l in range(L):
        s = scs[l].numpy()
        want = oracle.score(synth.bits(Xs[l]), parity.weights_to_oracle(weights[l]))
        assert np.abs(s - want).max() <= parity.SCORE_ATOL
        keep = oracle.keep_mask(s, tau, w, cu_arg)
        Kp, Vp, tab, ln, n_used = oracle.compact_paged(synth.bits(Ks[l]), synth.bits(Vs[l]), keep, P, n_pool, max_pages,
                                                       cu_seqlens=cu_arg, first_page=first[l], fill=fill)
        np.testing.assert_array_equal(lens[l].numpy(), ln)
        assert int(used[l].item()) == n_used
        np.testing.assert_array_equal(tabs[l].numpy(), tab)              # entries no list uses keep their -1
        np.testing.assert_array_equal(synth.bits(pools_k[l]), Kp)        # pages outside [first, first + used) keep their fill
        np.testing.assert_array_equal(synth.bits(pools_v[l]), Vp)
    # the one-layer paged call
    pk, pv = torch.full_like(pools_k[1], -5.0), torch.full_like(pools_v[1], -5.0)
    tab1, len1, used1 = torch.full_like(tabs[1], -1), torch.zeros_like(lens[1]), torch.zeros_like(used[1])
    binding.kvzap_prefill_fused_paged_host(ctx.handle, 1, Xs[1], Ks[1], Vs[1], cu_t, B, tau, w, pk, pv, P, first[1], tab1,
                                           len1, used1, None)
    assert torch.equal(len1, lens[1]) and torch.equal(used1, used[1])
    assert torch.equal(pk.view(torch.int16), pools_k[1].view(torch.int16)) and torch.equal(pv.view(torch.int16), pools_v[1].view(torch.int16))
    ctx.close()
