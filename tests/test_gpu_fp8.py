"""The 8-bit (E4M3) scoring path against the oracle: the first layer on the tensor cores' 8-bit path
with per-token and per-row scales, then GELU / second layer / mask / compaction as for bf16.
Tolerance as everywhere: 2e-2 absolute on the scores (E4M3 products are exact in fp32; the
accumulation order differs), masks equal outside that band, compaction bit-exact given the scores."""
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


def _fp8_case(d_model, hidden, H, T, seed):
    X = synth.hidden_states(T, d_model, seed)
    X8, sx = synth.quantize_e4m3(X)
    if hidden:
        W1, b1, W2, b2 = synth.mlp_weights(d_model, hidden, H, seed + 1, "cpu", 0.3)
    else:
        W1, b1 = synth.linear_weights(d_model, H, seed + 1, "cpu", 0.3)
        W2 = b2 = None
    W18, sw = synth.quantize_e4m3(W1)
    return X8, sx, W18, sw, b1, W2, b2


def _oracle_scores(oracle, case, hidden):
    X8, sx, W18, sw, b1, W2, b2 = case
    if hidden:
        return oracle.score_mlp_fp8(X8.numpy(), sx.numpy(), W18.numpy(), sw.numpy(), b1.numpy(), synth.bits(W2), b2.numpy())
    return oracle.score_linear_fp8(X8.numpy(), sx.numpy(), W18.numpy(), sw.numpy(), b1.numpy())


@pytest.mark.parametrize("d_model,hidden,T", [(256, 0, 1), (256, 0, 300), (1024, 0, 4097), (256, 64, 129), (512, 128, 1000),
                                              (256, 256, 257), (256, 512, 520), (256, 640, 200), (4096, 512, 260), (5120, 640, 130),
                                              (1024, 512, 20000)])
def test_fp8_scores_match_oracle(binding, oracle, d_model, hidden, T):
    H = 8
    ctx = binding.Kvzap(d_model, hidden, H, 64, 1, max_tokens=T)
    case = _fp8_case(d_model, hidden, H, T, seed=T + hidden)
    X8, sx, W18, sw, b1, W2, b2 = case
    binding.kvzap_set_weights_fp8(ctx.handle, 0, W18.cuda(), sw.cuda(), b1.cuda(), parity.dev(W2), parity.dev(b2))
    scores = torch.empty(T, H, dtype=torch.float32, device="cuda")
    binding.kvzap_score_fp8(ctx.handle, 0, X8.cuda(), sx.cuda(), scores)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    rows = np.arange(T) if T * max(hidden, 8) * d_model < 3e9 else np.unique(np.concatenate([[0, 127, 128, T - 1], np.random.default_rng(0).integers(0, T, 400)]))
    sub = tuple(t[rows] if i in (0, 1) else t for i, t in enumerate(case))
    want = _oracle_scores(oracle, sub, hidden)
    got = scores.cpu().numpy()[rows]
    assert np.isfinite(got).all()
    assert np.abs(got - want).max() <= parity.SCORE_ATOL
    # the bf16 calls refuse a layer that holds 8-bit weights
    with pytest.raises(binding.KvzapError) as ei:
        ctx.score(0, torch.zeros(1, d_model, dtype=torch.bfloat16, device="cuda"))
    assert ei.value.status == 6
    ctx.close()


@pytest.mark.parametrize("seq_lens,hidden", [([700], 0), ([37, 64, 5, 0, 300, 900], 128), ([33000], 256)])
def test_fp8_fused_prefill_matches_oracle(binding, oracle, seq_lens, hidden):
    d_model, H, D, tau, w = 512, 8, 64, 0.25, 32
    T, B = int(sum(seq_lens)), len(seq_lens)
    ctx = binding.Kvzap(d_model, hidden, H, D, 1, T, max_seqs=B)
    case = _fp8_case(d_model, hidden, H, T, seed=5 + hidden)
    X8, sx, W18, sw, b1, W2, b2 = case
    binding.kvzap_set_weights_fp8(ctx.handle, 0, W18.cuda(), sw.cuda(), b1.cuda(), parity.dev(W2), parity.dev(b2))
    K, V = synth.keys_values(H, T, D, seed=9)
    cu = synth.cu_seqlens(seq_lens)
    cu_dev = torch.from_numpy(cu).cuda() if B > 1 else None
    cu_arg = cu if B > 1 else None
    K_out, V_out = parity.poison_like(K).cuda(), parity.poison_like(V).cuda()
    lengths = torch.full((B, H), -1, dtype=torch.int32, device="cuda")
    scores = torch.empty(T, H, dtype=torch.float32, device="cuda")
    binding.kvzap_prefill_fused_fp8(ctx.handle, 0, X8.cuda(), sx.cuda(), parity.dev(K), parity.dev(V), cu_dev, B, tau, w,
                                    K_out, V_out, lengths, scores)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    want = _oracle_scores(oracle, case, hidden)
    s = scores.cpu().numpy()
    assert np.abs(s - want).max() <= parity.SCORE_ATOL
    parity.check_mask_band(oracle, s, want, tau, w, cu_arg)
    parity.check_compaction(oracle, K, V, s, tau, w, cu_arg, K_out.cpu(), V_out.cpu(), lengths)
    ctx.close()


@pytest.mark.parametrize("seq_lens,hidden,P", [([900], 128, 16), ([37, 0, 300, 129], 0, 4), ([20000], 640, 16)])
def test_fp8_fused_paged_prefill_matches_oracle(binding, oracle, seq_lens, hidden, P):
    """E4M3 hidden states into a paged output: scores against the 8-bit oracle, pools, page tables and lengths bit for bit
    against the oracle's paged compaction on the GPU's scores."""
    d_model, H, D, tau, w = 512, 8, 64, 0.25, 32
    T, B = int(sum(seq_lens)), len(seq_lens)
    ctx = binding.Kvzap(d_model, hidden, H, D, 1, T, max_seqs=B)
    case = _fp8_case(d_model, hidden, H, T, seed=11 + hidden)
    X8, sx, W18, sw, b1, W2, b2 = case
    binding.kvzap_set_weights_fp8(ctx.handle, 0, W18.cuda(), sw.cuda(), b1.cuda(), parity.dev(W2), parity.dev(b2))
    K, V = synth.keys_values(H, T, D, seed=12)
    cu = synth.cu_seqlens(seq_lens)
    cu_dev = torch.from_numpy(cu).cuda() if B > 1 else None
    cu_arg = cu if B > 1 else None
    n_pool, max_pages, first_page = H * (T // P + B + 1) + 5, max(seq_lens) // P + 2, 2
    pool = lambda: torch.full((n_pool, P, D), -5.0, dtype=torch.bfloat16, device="cuda")
    K_pool, V_pool = pool(), pool()
    table = torch.full((B * H, max_pages), -1, dtype=torch.int32, device="cuda")
    lengths = torch.zeros(B, H, dtype=torch.int32, device="cuda")
    used = torch.zeros(1, dtype=torch.int32, device="cuda")
    scores = torch.empty(T, H, dtype=torch.float32, device="cuda")
    binding.kvzap_prefill_fused_paged_fp8(ctx.handle, 0, X8.cuda(), sx.cuda(), parity.dev(K), parity.dev(V), cu_dev, B, tau, w,
                                          K_pool, V_pool, P, first_page, table, lengths, used, scores)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    want = _oracle_scores(oracle, case, hidden)
    s = scores.cpu().numpy()
    assert np.abs(s - want).max() <= parity.SCORE_ATOL
    keep = parity.check_mask_band(oracle, s, want, tau, w, cu_arg)
    fill = int(synth.bits(torch.tensor([-5.0], dtype=torch.bfloat16))[0])
    Kp, Vp, tab, ln, n_used = oracle.compact_paged(synth.bits(K), synth.bits(V), keep, P, n_pool, max_pages,
                                                   cu_seqlens=cu_arg, first_page=first_page, fill=fill)
    np.testing.assert_array_equal(lengths.cpu().numpy(), ln)
    assert int(used.item()) == n_used
    np.testing.assert_array_equal(table.cpu().numpy(), tab)
    np.testing.assert_array_equal(synth.bits(K_pool), Kp)
    np.testing.assert_array_equal(synth.bits(V_pool), Vp)
    ctx.close()


def _export(binding, ctx, cache, b, l, h, cap, D):
    K_out = torch.zeros(cap, D, dtype=torch.bfloat16, device="cuda")
    V_out = torch.zeros(cap, D, dtype=torch.bfloat16, device="cuda")
    n = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.kvzap_cache_export(ctx.handle, cache, b, l, h, K_out, V_out, n)
    torch.cuda.synchronize()
    n = int(n.item())
    return synth.bits(K_out)[:n], synth.bits(V_out)[:n], n


@pytest.mark.parametrize("d_model,hidden,w,P,B,L", [
    (256, 128, 8, 4, 3, 2),       # the one-launch step (four CTAs per tile, two halves of K)
    (512, 512, 16, 16, 5, 3),     # the same with 256 hidden units per slice
    (256, 64, 0, 4, 2, 2),        # no window: scoring launch, then the general update
    (256, 0, 5, 16, 2, 1),        # KVzap-Linear: layer after layer through the prefill kernel, then the update
    (256, 128, 8, 4, 130, 1),     # two token tiles per layer
])
def test_fp8_decode_steps_match_decode_oracle(binding, oracle, d_model, hidden, w, P, B, L):
    """kvzap_decode_step_fp8: scores against the 8-bit oracle, eviction decisions and list contents bit for bit
    against the decode oracle fed the GPU's scores."""
    H, D, tau, n_steps = 8, 64, 0.1, 30 if B < 100 else 14
    ctx = binding.Kvzap(d_model, hidden, H, D, L, max_tokens=max(B, 128), max_seqs=1)
    cases = []
    for l in range(L):
        case = _fp8_case(d_model, hidden, H, 1, seed=90 + l)        # weights of layer l (its one-token input is not used)
        cases.append(case)
        _, _, W18, sw, b1, W2, b2 = case
        binding.kvzap_set_weights_fp8(ctx.handle, l, W18.cuda(), sw.cuda(), b1.cuda(),
                                      parity.dev(W2) if W2 is not None else None, parity.dev(b2) if b2 is not None else None)
    max_pages = n_steps // P + 2
    n_pool = B * L * H * max_pages
    K_pool = torch.zeros(n_pool, P, D, dtype=torch.bfloat16, device="cuda")
    V_pool = torch.zeros_like(K_pool)
    cache = binding.kvzap_cache_create(ctx.handle, B, w, P, K_pool, V_pool, max_pages)
    dec = oracle.DecodeOracle(B, L, H, D, w)
    worst = 0.0
    for step in range(n_steps):
        X = synth.hidden_states(L * B, d_model, seed=1500 + step)
        X8, sx = synth.quantize_e4m3(X)
        if step % 3 == 2:
            sx = None                                          # NULL scales = 1
        K_new, V_new = synth.keys_values(L * B, H, D, seed=2500 + step)
        K_new, V_new = K_new.view(L, B, H, D), V_new.view(L, B, H, D)
        scores = torch.empty(L, B, H, dtype=torch.float32, device="cuda")
        binding.kvzap_decode_step_fp8(ctx.handle, cache, 0, L, X8.cuda().view(L, B, d_model),
                                      sx.cuda().view(L, B) if sx is not None else None, parity.dev(K_new), parity.dev(V_new),
                                      tau, scores)
        torch.cuda.synchronize()
        s = scores.cpu().numpy()
        X8n = X8.numpy().reshape(L, B, d_model)
        sxn = sx.numpy().reshape(L, B) if sx is not None else np.ones((L, B), dtype=np.float32)
        for l in range(L):
            _, _, W18, sw, b1, W2, b2 = cases[l]
            if hidden:
                want = oracle.score_mlp_fp8(X8n[l], sxn[l], W18.numpy(), sw.numpy(), b1.numpy(), synth.bits(W2), b2.numpy())
            else:
                want = oracle.score_linear_fp8(X8n[l], sxn[l], W18.numpy(), sw.numpy(), b1.numpy())
            worst = max(worst, float(np.abs(s[l] - want).max()))
            Kb, Vb = synth.bits(K_new[l]), synth.bits(V_new[l])
            for b in range(B):
                dec.append(b, l, s[l, b], Kb[b], Vb[b], tau)
    assert worst <= parity.SCORE_ATOL, worst
    assert ctx.poll_status() == 0
    lists = [(b, l, h) for b in range(B) for l in range(L) for h in range(H)] if B < 100 else \
            [(0, 0, 0), (127, 0, 3), (129, 0, 7), (64, 0, 5)]
    for b, l, h in lists:
        _pos, Kd, Vd = dec.logical(b, l, h)
        Kg, Vg, n = _export(binding, ctx, cache, b, l, h, n_steps + 1, D)
        assert n == len(Kd), (b, l, h)
        np.testing.assert_array_equal(Kg, Kd)
        np.testing.assert_array_equal(Vg, Vd)
    binding.kvzap_cache_destroy(cache)
    ctx.close()


def test_fp8_decode_steps_captured_in_a_cuda_graph(binding, oracle):
    """Two 8-bit decode steps captured once and replayed with refilled static buffers: scores against the 8-bit
    oracle, lists bit for bit against the decode oracle."""
    d_model, hidden, H, D, w, P, B, L, tau, n_replays = 256, 128, 8, 64, 8, 4, 6, 2, 0.1, 8
    ctx = binding.Kvzap(d_model, hidden, H, D, L, max_tokens=128, max_seqs=1, trusted_producers=True)
    cases = []
    for l in range(L):
        case = _fp8_case(d_model, hidden, H, 1, seed=190 + l)
        cases.append(case)
        _, _, W18, sw, b1, W2, b2 = case
        binding.kvzap_set_weights_fp8(ctx.handle, l, W18.cuda(), sw.cuda(), b1.cuda(), parity.dev(W2), parity.dev(b2))
    n_steps = 2 * n_replays + 2
    max_pages = n_steps // P + 2
    n_pool = B * L * H * max_pages
    K_pool = torch.zeros(n_pool, P, D, dtype=torch.bfloat16, device="cuda")
    V_pool = torch.zeros_like(K_pool)
    cache = binding.kvzap_cache_create(ctx.handle, B, w, P, K_pool, V_pool, max_pages)
    dec = oracle.DecodeOracle(B, L, H, D, w)
    X8 = [torch.zeros(L, B, d_model, dtype=torch.uint8, device="cuda") for _ in range(2)]
    SX = [torch.zeros(L, B, dtype=torch.float32, device="cuda") for _ in range(2)]
    Kn = [torch.zeros(L, B, H, D, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    Vn = [torch.zeros(L, B, H, D, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    sc = [torch.zeros(L, B, H, dtype=torch.float32, device="cuda") for _ in range(2)]
    feed = {}

    def fill(i, step):
        x8, sx = synth.quantize_e4m3(synth.hidden_states(L * B, d_model, seed=3500 + step))
        k, v = synth.keys_values(L * B, H, D, seed=4500 + step)
        X8[i].copy_(x8.view(L, B, d_model)); SX[i].copy_(sx.view(L, B)); Kn[i].copy_(k.view(L, B, H, D)); Vn[i].copy_(v.view(L, B, H, D))
        feed[i] = (x8.numpy().reshape(L, B, d_model), sx.numpy().reshape(L, B), synth.bits(k.view(L, B, H, D)), synth.bits(v.view(L, B, H, D)))

    def iteration():
        for i in range(2):
            binding.kvzap_decode_step_fp8(ctx.handle, cache, 0, L, X8[i], SX[i], Kn[i], Vn[i], tau, sc[i])

    worst = [0.0]

    def account():
        assert ctx.poll_status() == 0
        for i in range(2):
            s = sc[i].cpu().numpy()
            x8, sx, kb, vb = feed[i]
            for l in range(L):
                _, _, W18, sw, b1, W2, b2 = cases[l]
                want = oracle.score_mlp_fp8(x8[l], sx[l], W18.numpy(), sw.numpy(), b1.numpy(), synth.bits(W2), b2.numpy())
                worst[0] = max(worst[0], float(np.abs(s[l] - want).max()))
                for b in range(B):
                    dec.append(b, l, s[l, b], kb[l, b], vb[l, b], tau)

    fill(0, 0); fill(1, 1)
    iteration()
    torch.cuda.synchronize()
    account()
    graph = torch.cuda.CUDAGraph()
    fill(0, 2); fill(1, 3)
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=torch.cuda.Stream()):
        iteration()
    for r in range(n_replays):
        if r > 0:
            fill(0, 2 + 2 * r); fill(1, 3 + 2 * r)
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        account()
    assert worst[0] <= parity.SCORE_ATOL, worst[0]
    for b in range(B):
        for l in range(L):
            for h in range(H):
                _pos, Kd, Vd = dec.logical(b, l, h)
                Kg, Vg, n = _export(binding, ctx, cache, b, l, h, n_steps + 1, D)
                assert n == len(Kd), (b, l, h)
                np.testing.assert_array_equal(Kg, Kd)
                np.testing.assert_array_equal(Vg, Vd)
    binding.kvzap_cache_destroy(cache)
    ctx.close()


def test_fp8_needs_d_model_multiple_of_128_and_its_own_weights(binding):
    ctx = binding.Kvzap(192, 0, 8, 64, 1, max_tokens=64)
    W = torch.zeros(8, 192, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.KvzapError) as ei:
        binding.kvzap_set_weights_fp8(ctx.handle, 0, W, None)
    assert ei.value.status == 2
    ctx.close()
    ctx = binding.Kvzap(256, 0, 8, 64, 1, max_tokens=64)
    ctx.set_weights(0, *[t.cuda() for t in synth.linear_weights(256, 8, 1)])
    with pytest.raises(binding.KvzapError) as ei:
        binding.kvzap_score_fp8(ctx.handle, 0, torch.zeros(4, 256, dtype=torch.uint8, device="cuda"), None,
                                torch.zeros(4, 8, device="cuda"))
    assert ei.value.status == 6
    ctx.close()
