"""The decode loop captured in a CUDA graph and replayed.

A serving loop that captures its decode iteration once and replays it must get, from every replay, what the same calls
enqueued one by one give: a one-launch decode step learns its step number on the device (a ticket drawn by each CTA),
so nothing that changes from step to step is baked into the captured launch.  The test captures two steps, each
followed by the attention over the lists it leaves (inputs and outputs in static buffers, refilled before every replay),
replays the graph many times and replays the same token stream through the decode oracle: scores within the
tolerance, attention outputs against the oracle's lists, every list bit for bit at the end.
"""
import numpy as np
import pytest
import torch

from paper_2601_07891_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu

ATTN_ATOL = 2e-2


@pytest.fixture(scope="module")
def binding():
    from paper_2601_07891_b200 import binding as b
    b.load()
    return b


def _export(binding, ctx, cache, b, l, h, cap, D):
    K_out = torch.zeros(cap, D, dtype=torch.bfloat16, device="cuda")
    V_out = torch.zeros(cap, D, dtype=torch.bfloat16, device="cuda")
    n = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.kvzap_cache_export(ctx.handle, cache, b, l, h, K_out, V_out, n)
    torch.cuda.synchronize()
    n = int(n.item())
    return synth.bits(K_out)[:n], synth.bits(V_out)[:n], n


@pytest.mark.parametrize("hidden,L,B,trusted", [(128, 3, 5, True), (512, 2, 130, True), (128, 2, 4, False)])
def test_captured_decode_steps_replay_like_single_calls(binding, oracle, hidden, L, B, trusted):
    d_model, H, D, w, P, G, tau, n_replays = 256, 8, 64, 16, 16, 4, 0.05, 20
    n_steps = 2 * n_replays + 2
    ctx = binding.Kvzap(d_model, hidden, H, D, L, max_tokens=max(B, 128), max_seqs=1, trusted_producers=trusted)
    wts = [synth.mlp_weights(d_model, hidden, H, 40 + l, "cpu", 0.3) for l in range(L)]
    for l in range(L):
        ctx.set_weights(l, *[parity.dev(x) for x in wts[l]])
    max_pages = n_steps // P + 2
    n_pool = B * L * H * max_pages
    K_pool = torch.full((n_pool, P, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    V_pool = torch.full_like(K_pool, float("nan"))
    cache = binding.kvzap_cache_create(ctx.handle, B, w, P, K_pool, V_pool, max_pages)
    dec = oracle.DecodeOracle(B, L, H, D, w)
    # static buffers of the captured iteration (two steps)
    X = [torch.zeros(L, B, d_model, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    Kn = [torch.zeros(L, B, H, D, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    Vn = [torch.zeros(L, B, H, D, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    sc = [torch.zeros(L, B, H, dtype=torch.float32, device="cuda") for _ in range(2)]
    Q = [torch.zeros(L, B, H * G, D, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    O = [torch.zeros(L, B, H * G, D, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    scale = 1.0 / np.sqrt(D)
    feed = {}

    def fill(i, step):
        x = synth.hidden_states(L * B, d_model, seed=7000 + step).view(L, B, d_model)
        k, v = synth.keys_values(L * B, H, D, seed=8000 + step)
        q = synth.hidden_states(L * B * H * G, D, seed=9000 + step).view(L, B, H * G, D)
        X[i].copy_(x); Kn[i].copy_(k.view(L, B, H, D)); Vn[i].copy_(v.view(L, B, H, D)); Q[i].copy_(q)
        feed[i] = (synth.bits(x), synth.bits(k.view(L, B, H, D)), synth.bits(v.view(L, B, H, D)), synth.bits(q))

    def iteration():
        for i in range(2):
            binding.kvzap_decode_step(ctx.handle, cache, 0, L, X[i], Kn[i], Vn[i], tau, sc[i])
            binding.kvzap_decode_attention(ctx.handle, cache, 0, L, Q[i], scale, O[i])

    worst_s, worst_o = [0.0], [0.0]

    def account(first_step):
        s_all = [t.cpu().numpy() for t in sc]
        o_all = [t.float().cpu().numpy() for t in O]
        assert ctx.poll_status() == 0
        for i in range(2):
            xb, kb, vb, qb = feed[i]
            for l in range(L):
                want = oracle.score(xb[l], parity.weights_to_oracle(wts[l]))
                worst_s[0] = max(worst_s[0], float(np.abs(s_all[i][l] - want).max()))
                for b in range(B):
                    dec.append(b, l, s_all[i][l, b], kb[l, b], vb[l, b], tau)
            if i == 1:      # the attention behind the second step sees the lists as they are now
                for l in range(L):
                    for b in range(0, B, max(1, B // 4)):
                        for h in (0, H - 1):
                            _pos, Kd, Vd = dec.logical(b, l, h)
                            want = oracle.attention(qb[l, b, h * G:(h + 1) * G], Kd, Vd, scale)
                            worst_o[0] = max(worst_o[0], float(np.abs(o_all[i][l, b, h * G:(h + 1) * G] - want).max()))

    # one iteration enqueued call by call (also builds whatever the calls build on first use), then the capture
    fill(0, 0); fill(1, 1)
    iteration()
    torch.cuda.synchronize()
    account(0)
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    fill(0, 2); fill(1, 3)
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=side):
        iteration()
    # the capture itself ran nothing
    for r in range(n_replays):
        if r > 0:
            fill(0, 2 + 2 * r); fill(1, 3 + 2 * r)
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        account(2 + 2 * r)
    assert worst_s[0] <= parity.SCORE_ATOL, worst_s[0]
    assert worst_o[0] <= ATTN_ATOL, worst_o[0]
    lists = [(b, l, h) for b in range(B) for l in range(L) for h in range(H)] if B < 100 else \
            [(0, 0, 0), (127, 1, 3), (129, 0, 7), (64, 1, 5)]
    for b, l, h in lists:
        _pos, Kd, Vd = dec.logical(b, l, h)
        Kg, Vg, n = _export(binding, ctx, cache, b, l, h, n_steps + 1, D)
        assert n == len(Kd), (b, l, h)
        np.testing.assert_array_equal(Kg, Kd)
        np.testing.assert_array_equal(Vg, Vd)
    binding.kvzap_cache_destroy(cache)
    ctx.close()
