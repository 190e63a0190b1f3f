"""GPU parity for kvzap_prefill_to_cache_batch: several prompts (or chunks of prompts) into several sequence
slots of a decode cache in one call.

Every sequence must end up exactly as a prefill of its whole prompt leaves it (Algorithm 1 on the concatenation,
per sequence): each list is exported and compared bit for bit with the oracle's compaction on the GPU's own scores,
after each round of chunks and after decode steps on top; page tables are checked for validity (no page owned
twice), since which pages a list gets depends on the allocation order.
"""
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
    if hidden == 0:
        return synth.linear_weights(d_model, H, seed, "cpu", 0.3)
    return synth.mlp_weights(d_model, hidden, H, seed, "cpu", 0.3)


def _export(binding, ctx, cache, b, l, h, cap, D):
    K_out = torch.zeros(cap, D, dtype=torch.bfloat16, device="cuda")
    V_out = torch.zeros(cap, D, dtype=torch.bfloat16, device="cuda")
    n = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.kvzap_cache_export(ctx.handle, cache, b, l, h, K_out, V_out, n)
    torch.cuda.synchronize()
    n = int(n.item())
    return synth.bits(K_out)[:n], synth.bits(V_out)[:n], n


@pytest.mark.parametrize("hidden,w,P,L,rounds", [
    # rounds: per call, {slot: chunk length}; slots out of order, not consecutive, not all in every call
    (128, 16, 16, 2, [{5: 300, 0: 70, 3: 1}, {3: 200, 5: 9}, {0: 130, 2: 40, 5: 33}]),
    (0, 8, 4, 1, [{1: 50, 4: 5}, {4: 5, 1: 3}, {4: 120}]),                      # chunks shorter than the window
    (64, 0, 16, 1, [{0: 100, 1: 17}, {1: 90, 2: 260}]),                         # no window
    (128, 128, 16, 1, [{2: 1000, 0: 100}, {0: 100, 1: 129, 2: 24}]),            # w = 128: a chunk inside one window
])
def test_batched_prompts_equal_whole_prompt_prefill_per_sequence(binding, oracle, hidden, w, P, L, rounds):
    d_model, H, D, tau, n_slots, k = 256, 8, 64, 0.1, 6, 5
    total = {}
    for r in rounds:
        for slot, m in r.items():
            total[slot] = total.get(slot, 0) + m
    cap = max(total.values()) + k
    max_call = max(sum(r.values()) for r in rounds)
    ctx = binding.Kvzap(d_model, hidden, H, D, L, max_tokens=max(max_call, n_slots), max_seqs=n_slots)
    wts = [_weights(d_model, hidden, H, seed=300 + l) for l in range(L)]
    for l in range(L):
        ctx.set_weights(l, *[parity.dev(x) for x in wts[l]])
    max_pages = cap // P + 2
    n_pool = n_slots * L * H * max_pages
    K_pool = torch.full((n_pool, P, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    V_pool = torch.full_like(K_pool, float("nan"))
    cache = binding.kvzap_cache_create(ctx.handle, n_slots, w, P, K_pool, V_pool, max_pages)
    # per (slot, layer): everything fed so far
    Xs = {(s, l): [] for s in total for l in range(L)}
    Ks = {(s, l): [] for s in total for l in range(L)}
    Vs = {(s, l): [] for s in total for l in range(L)}
    Ss = {(s, l): [] for s in total for l in range(L)}
    seed = 0

    def check(slots):
        torch.cuda.synchronize()
        assert ctx.poll_status() == 0
        for s in slots:
            for l in range(L):
                if not Ks[(s, l)]:
                    continue
                K = np.concatenate(Ks[(s, l)], axis=1)
                V = np.concatenate(Vs[(s, l)], axis=1)
                sc = np.concatenate(Ss[(s, l)], axis=0)
                want = oracle.score(np.concatenate(Xs[(s, l)], axis=0), parity.weights_to_oracle(wts[l]))
                assert np.abs(sc - want).max() <= parity.SCORE_ATOL
                keep = oracle.keep_mask(sc, tau, w)
                Kc, Vc, ln = oracle.compact(K, V, keep)
                for h in range(H):
                    Kg, Vg, n = _export(binding, ctx, cache, s, l, h, cap, D)
                    assert n == ln[0, h], (s, l, h)
                    np.testing.assert_array_equal(Kg, Kc[h, :n])
                    np.testing.assert_array_equal(Vg, Vc[h, :n])

    for r in rounds:
        slots = list(r.keys())
        lens = [r[s] for s in slots]
        cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]).astype(np.int32), device="cuda")
        n_tok = int(sum(lens))
        for l in range(L):
            seed += 1
            X = synth.hidden_states(n_tok, d_model, seed=seed)
            K, V = synth.keys_values(H, n_tok, D, seed=seed + 7000)
            sc = torch.empty(n_tok, H, dtype=torch.float32, device="cuda")
            binding.kvzap_prefill_to_cache_batch(ctx.handle, cache, l, slots, cu, parity.dev(X), parity.dev(K), parity.dev(V), tau, sc)
            torch.cuda.synchronize()
            s_np, Xb, Kb, Vb = sc.cpu().numpy(), synth.bits(X), synth.bits(K), synth.bits(V)
            t = 0
            for s, m in zip(slots, lens):
                Xs[(s, l)].append(Xb[t:t + m]); Ks[(s, l)].append(Kb[:, t:t + m]); Vs[(s, l)].append(Vb[:, t:t + m])
                Ss[(s, l)].append(s_np[t:t + m])
                t += m
        check(slots)
    # decode steps on top: all slots step together (slots that never got a prompt are inactive and stay empty)
    for step in range(k):
        seed += 1
        X = synth.hidden_states(L * n_slots, d_model, seed=seed).view(L, n_slots, d_model)
        Kn, Vn = synth.keys_values(L * n_slots, H, D, seed=seed + 7000)
        Kn, Vn = Kn.view(L, n_slots, H, D), Vn.view(L, n_slots, H, D)
        sc = torch.empty(L, n_slots, H, dtype=torch.float32, device="cuda")
        binding.kvzap_decode_step(ctx.handle, cache, 0, L, parity.dev(X), parity.dev(Kn), parity.dev(Vn), tau, sc)
        torch.cuda.synchronize()
        s_np, Xb, Kb, Vb = sc.cpu().numpy(), synth.bits(X), synth.bits(Kn), synth.bits(Vn)
        for s in total:
            for l in range(L):
                Xs[(s, l)].append(Xb[l, s][None]); Ks[(s, l)].append(Kb[l, s][:, None]); Vs[(s, l)].append(Vb[l, s][:, None])
                Ss[(s, l)].append(s_np[l, s][None])
    check(list(total.keys()))
    # page tables: every page of every list is in range and owned once
    n_lists = n_slots * L * H
    prefix = torch.zeros(n_lists, dtype=torch.int32, device="cuda")
    table = torch.zeros(n_lists, max_pages, dtype=torch.int32, device="cuda")
    nxt = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.kvzap_cache_snapshot(ctx.handle, cache, prefix, table, nxt)
    torch.cuda.synchronize()
    pl, tb = prefix.cpu().numpy(), table.cpu().numpy()
    owned = []
    for li in range(n_lists):
        owned += tb[li, :(pl[li] + P - 1) // P].tolist()
    assert len(owned) == len(set(owned)) and all(0 <= p < n_pool for p in owned)
    binding.kvzap_cache_destroy(cache)
    ctx.close()


def test_batched_prompts_argument_checks(binding):
    d_model, H, D = 256, 8, 64
    ctx = binding.Kvzap(d_model, 0, H, D, 1, max_tokens=64, max_seqs=4)
    W, b = synth.linear_weights(d_model, H, 1)
    ctx.set_weights(0, parity.dev(W), parity.dev(b))
    pool = torch.zeros(64, 16, D, dtype=torch.bfloat16, device="cuda")
    cache = binding.kvzap_cache_create(ctx.handle, 4, 16, 16, pool, pool.clone(), 2)
    X = parity.dev(synth.hidden_states(20, d_model, seed=1))
    K, V = [parity.dev(t) for t in synth.keys_values(H, 20, D, seed=2)]
    sc = torch.empty(20, H, dtype=torch.float32, device="cuda")
    cu = torch.tensor([0, 10, 20], dtype=torch.int32, device="cuda")
    with pytest.raises(binding.KvzapError):
        binding.kvzap_prefill_to_cache_batch(ctx.handle, cache, 0, [1, 1], cu, X, K, V, 0.0, sc)     # a slot twice
    with pytest.raises(binding.KvzapError):
        binding.kvzap_prefill_to_cache_batch(ctx.handle, cache, 0, [0, 4], cu, X, K, V, 0.0, sc)     # slot out of range
    with pytest.raises(binding.KvzapError):
        binding.kvzap_prefill_to_cache_batch(ctx.handle, cache, 1, [0, 1], cu, X, K, V, 0.0, sc)     # layer out of range
    binding.kvzap_prefill_to_cache_batch(ctx.handle, cache, 0, [3, 0], cu, X, K, V, 0.0, sc)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    lengths = torch.zeros(4, 1, H, dtype=torch.int32, device="cuda")
    binding.kvzap_cache_lengths(ctx.handle, cache, lengths)
    torch.cuda.synchronize()
    ln = lengths.cpu().numpy()
    assert (ln[1] == 0).all() and (ln[2] == 0).all() and (ln[0] == 10).all() and (ln[3] == 10).all()   # w = 16 > 10: all kept
    binding.kvzap_cache_destroy(cache)
    ctx.close()
