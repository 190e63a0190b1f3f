"""The object layer of the binding (Kvzap / KvzapCache) does argument marshalling only: the same calls
through it give the same bits as through the functions, and the usage shown in the README runs."""
import numpy as np
import pytest
import torch

from paper_2601_07891_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu


def test_prefill_chunks_decode_and_attention_through_the_objects(oracle):
    from paper_2601_07891_b200 import binding
    d_model, hidden, H, D, L, G, w, P, tau = 256, 128, 8, 64, 2, 4, 16, 16, 0.1
    T0, k = 200, 6
    ctx = binding.Kvzap(d_model, hidden, H, D, L, max_tokens=256)
    weights = [synth.mlp_weights(d_model, hidden, H, 40 + l, "cpu", 0.3) for l in range(L)]
    for l in range(L):
        ctx.set_weights(l, *[parity.dev(x) for x in weights[l]])
    n_pool = L * H * ((T0 + k) // P + 2)
    K_pool = torch.zeros(n_pool, P, D, dtype=torch.bfloat16, device="cuda")
    V_pool = torch.zeros_like(K_pool)
    cache = ctx.create_cache(1, w, P, K_pool, V_pool, (T0 + k) // P + 2)
    dec = oracle.DecodeOracle(1, L, H, D, w)
    Xs = [synth.hidden_states(T0 + k, d_model, seed=60 + l) for l in range(L)]
    KVs = [synth.keys_values(H, T0 + k, D, seed=70 + l) for l in range(L)]
    # the prompt in two chunks per layer
    for l in range(L):
        for a, b in ((0, 120), (120, T0)):
            s = cache.prefill(l, 0, parity.dev(Xs[l][a:b]), parity.dev(KVs[l][0][:, a:b].contiguous()),
                              parity.dev(KVs[l][1][:, a:b].contiguous()), tau)
            s = s.cpu().numpy()
            Kb, Vb = synth.bits(KVs[l][0]), synth.bits(KVs[l][1])
            for t in range(a, b):
                dec.append(0, l, s[t - a], Kb[:, t], Vb[:, t], tau)
    # decode steps, each followed by attention
    for t in range(T0, T0 + k):
        X = torch.stack([Xs[l][t] for l in range(L)]).view(L, 1, d_model)
        Kn = torch.stack([KVs[l][0][:, t] for l in range(L)]).view(L, 1, H, D)
        Vn = torch.stack([KVs[l][1][:, t] for l in range(L)]).view(L, 1, H, D)
        sc = torch.empty(L, 1, H, dtype=torch.float32, device="cuda")
        cache.decode_step(0, L, parity.dev(X), parity.dev(Kn), parity.dev(Vn), tau, sc)
        Q = synth.hidden_states(L * H * G, D, seed=500 + t).view(L, 1, H * G, D)
        O = cache.attention(0, L, parity.dev(Q))
        torch.cuda.synchronize()
        s = sc.cpu().numpy()
        for l in range(L):
            dec.append(0, l, s[l, 0], synth.bits(Kn)[l, 0], synth.bits(Vn)[l, 0], tau)
        got = O.float().cpu().numpy()
        for l in range(L):
            for h in range(H):
                _pos, Kd, Vd = dec.logical(0, l, h)
                want = oracle.attention(synth.bits(Q)[l, 0, h * G:(h + 1) * G], Kd, Vd, 1.0 / np.sqrt(D))
                assert np.abs(got[l, 0, h * G:(h + 1) * G] - want).max() <= 2e-2
    assert ctx.poll_status() == 0
    ln = cache.lengths().cpu().numpy()
    for l in range(L):
        for h in range(H):
            assert ln[0, l, h] == dec.length(0, l, h)
    cache.close()
    ctx.close()


def test_write_side_and_topk_methods_match_the_function_calls(oracle):
    from paper_2601_07891_b200 import binding
    d_model, H, D, T, w = 256, 8, 64, 500, 16
    ctx = binding.Kvzap(d_model, 0, H, D, 1, T)
    W, b = synth.linear_weights(d_model, H, 5, "cpu", 0.3)
    ctx.set_weights(0, parity.dev(W), parity.dev(b))
    X = parity.dev(synth.hidden_states(T, d_model, seed=1))
    K, V = synth.keys_values(H, T, D, seed=2)
    K, V = parity.dev(K), parity.dev(V)
    K1, V1, len1 = ctx.prefill_fused(0, X, K, V, 0.2, w)
    K2, V2, len2 = ctx.prefill_write(0, X, K.transpose(0, 1).contiguous(), V.transpose(0, 1).contiguous(), 0.2, w)
    torch.cuda.synchronize()
    n = len1.cpu().numpy()[0]
    assert torch.equal(len1, len2)
    for h in range(H):
        assert torch.equal(K1[h, :n[h]].view(torch.int16), K2[h, :n[h]].view(torch.int16))
        assert torch.equal(V1[h, :n[h]].view(torch.int16), V2[h, :n[h]].view(torch.int16))
    s = ctx.score(0, X)
    tau = torch.empty(1, H, dtype=torch.float32, device="cuda")
    K3, V3, len3 = ctx.prune_prefill_topk(K, V, s, 0.25, w, tau_out=tau)
    torch.cuda.synchronize()
    keep, tau_ref = oracle.topk_mask(s.cpu().numpy(), 0.25, w)
    np.testing.assert_array_equal(tau.cpu().numpy(), tau_ref)
    np.testing.assert_array_equal(len3.cpu().numpy()[0], keep.sum(1))
    ctx.close()
