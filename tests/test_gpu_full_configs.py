"""GPU parity at the full sizes of the five benchmark configurations (one layer each),
in the launch configuration bench.py times.

Where the oracle cannot score every token in seconds (MLP at 32k / 128k tokens), scores
are compared on sampled rows (first and last tile, tile seams, random rows) -- scoring is
independent per position -- while mask, lengths and compacted rows are always checked in
full, bit for bit, against the oracle run on the GPU's own scores.
"""
import numpy as np
import pytest
import torch

from paper_2601_07891_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu

W = synth.WORKLOADS


@pytest.fixture(scope="module")
def binding():
    from paper_2601_07891_b200 import binding as b
    b.load()
    return b


def _sample_rows(T, n, seed):
    rng = np.random.default_rng(seed)
    fixed = [0, 1, 127, 128, 129, T // 2 - 1, T // 2, T - 130, T - 129, T - 128, T - 2, T - 1]
    rows = np.unique(np.concatenate([np.array([r for r in fixed if 0 <= r < T]), rng.integers(0, T, n)]))
    return rows.astype(np.int64)


def _prefill_case(binding, oracle, wl, layer, tau, sample=None, seed_shift=0):
    dev = "cuda"
    B, T = wl.batch, wl.seq_len
    n_tokens, H, D = B * T, wl.n_kv_heads, wl.head_dim
    ctx = binding.Kvzap(wl.d_model, wl.hidden, H, D, 1, n_tokens, max_seqs=B, trusted_producers=True)
    weights = synth.surrogate_weights(wl, layer, dev)
    ctx.set_weights(0, *weights)
    X = synth.hidden_states(n_tokens, wl.d_model, 31 + layer + seed_shift, dev, wl.token_scale_sigma)
    K, V = synth.keys_values(H, n_tokens, D, 32 + layer + seed_shift, dev)
    cu = synth.cu_seqlens([T] * B)
    cu_dev = torch.from_numpy(cu).cuda() if B > 1 else None
    cu_arg = cu if B > 1 else None
    scores = torch.empty(n_tokens, H, dtype=torch.float32, device=dev)
    out = dict(ctx=ctx, X=X, K=K, V=V, cu=cu_arg, cu_dev=cu_dev, scores=scores, weights=weights)
    return out


def _check_scores_sampled(oracle, case, sample, seed):
    X, scores = case["X"], case["scores"]
    T = X.shape[0]
    rows = np.arange(T) if sample is None else _sample_rows(T, sample, seed)
    rows_t = torch.from_numpy(rows).cuda()
    Xs = X.index_select(0, rows_t).cpu()
    got = scores.index_select(0, rows_t).cpu().numpy()
    want = oracle.score(synth.bits(Xs), parity.weights_to_oracle(tuple(w.cpu() for w in case["weights"])))
    err = float(np.abs(got - want).max())
    assert err <= parity.SCORE_ATOL, err
    return rows, got, want


def _dense_prune_and_check(binding, oracle, case, wl, tau, sample, seed):
    ctx, X, K, V = case["ctx"], case["X"], case["K"], case["V"]
    K_out, V_out = parity.poison_like(K), parity.poison_like(V)
    _, _, lengths = ctx.prefill_fused(0, X, K, V, tau, wl.window, cu_seqlens=case["cu_dev"], K_out=K_out, V_out=V_out,
                                      scores_out=case["scores"])
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    rows, got, want = _check_scores_sampled(oracle, case, sample, seed)
    s = case["scores"].cpu().numpy()
    # mask: outside the tolerance band the GPU's decision equals the oracle's (on the sampled rows)
    keep_gpu_rows = (s[rows] >= np.float32(tau))
    keep_ref_rows = (want >= np.float32(tau))
    near = np.abs(want - np.float32(tau)) <= parity.SCORE_ATOL
    assert not ((keep_gpu_rows != keep_ref_rows) & ~near).any()
    keep, len_ref = parity.check_compaction(oracle, K.cpu(), V.cpu(), s, tau, wl.window, case["cu"], K_out.cpu(),
                                            V_out.cpu(), lengths)
    return keep, len_ref


def test_config1_linear_4k_full(binding, oracle):
    wl = W["linear_4k"]
    case = _prefill_case(binding, oracle, wl, 0, wl.tau)
    keep, lengths = _dense_prune_and_check(binding, oracle, case, wl, wl.tau, None, 1)
    frac = lengths.sum() / (wl.n_kv_heads * wl.seq_len)
    assert 0.30 < frac < 0.41          # about one third kept, plus the window
    case["ctx"].close()


def test_config2_qwen3_8b_mlp_32k_one_layer(binding, oracle):
    wl = W["qwen3_8b_prefill_32k"]
    case = _prefill_case(binding, oracle, wl, 3, wl.tau)
    keep, lengths = _dense_prune_and_check(binding, oracle, case, wl, wl.tau, 600, 2)
    assert (lengths >= wl.window).all()
    case["ctx"].close()


@pytest.mark.parametrize("tau", [0.0, 0.43, 0.84])
def test_config3_llama_linear_4x16k_one_layer(binding, oracle, tau):
    wl = W["llama31_8b_prefill_4x16k"]
    case = _prefill_case(binding, oracle, wl, 5, tau)
    keep, lengths = _dense_prune_and_check(binding, oracle, case, wl, tau, None, 3)
    assert lengths.shape == (4, 8) and (lengths >= wl.window).all()
    # each sequence's window is kept: last w positions of every sequence, every head
    T = wl.seq_len
    for b in range(wl.batch):
        assert keep[:, (b + 1) * T - wl.window:(b + 1) * T].all()
    case["ctx"].close()


def test_config4_qwen3_32b_mlp_128k_paged_one_layer(binding, oracle):
    wl = W["qwen3_32b_prefill_128k_paged"]
    case = _prefill_case(binding, oracle, wl, 7, wl.tau)
    ctx, X, K, V = case["ctx"], case["X"], case["K"], case["V"]
    H, D, T, P = wl.n_kv_heads, wl.head_dim, wl.seq_len, wl.page_tokens
    max_pages = T // P + 1
    n_pool = 45000                                   # 4 KiB pages: 176 MiB per pool
    K_pool = torch.full((n_pool, P, D), -5.0, dtype=torch.bfloat16, device="cuda")
    V_pool = torch.full((n_pool, P, D), -5.0, dtype=torch.bfloat16, device="cuda")
    table = torch.full((H, max_pages), -1, dtype=torch.int32, device="cuda")
    lengths = torch.zeros(1, H, dtype=torch.int32, device="cuda")
    used = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.kvzap_prefill_fused_paged(ctx.handle, 0, X, K, V, None, 1, wl.tau, wl.window, K_pool, V_pool, P, 0, table,
                                      lengths, used, case["scores"])
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    _check_scores_sampled(oracle, case, 300, 4)
    s = case["scores"].cpu().numpy()
    keep = oracle.keep_mask(s, wl.tau, wl.window)
    fill = int(synth.bits(torch.tensor([-5.0], dtype=torch.bfloat16))[0])
    Kp, Vp, tab, ln, n_used = oracle.compact_paged(synth.bits(K), synth.bits(V), keep, P, n_pool, max_pages, fill=fill)
    np.testing.assert_array_equal(lengths.cpu().numpy(), ln)
    assert int(used.item()) == n_used
    np.testing.assert_array_equal(table.cpu().numpy(), tab)
    np.testing.assert_array_equal(synth.bits(K_pool), Kp)
    np.testing.assert_array_equal(synth.bits(V_pool), Vp)
    ctx.close()


def test_config5_decode_b128_all_layers(binding, oracle):
    """36 layers x 128 sequences, w = 128, 16-token pages, 132 steps so that tokens leave the window.
    All steps are enqueued back to back with no host synchronisation in between and with a different
    scores buffer per step -- the launch configuration bench.py times, in which consecutive steps
    overlap on the GPU.  Scores: compared with the oracle on a few (step, layer) pairs.  Evictions and
    list contents: the decode oracle replays the GPU's own scores for a sample of lists."""
    wl = W["qwen3_8b_decode_b128"]
    L, B, H, D, w, P = wl.n_layers, wl.batch, wl.n_kv_heads, wl.head_dim, wl.window, wl.page_tokens
    n_steps = w + 4
    ctx = binding.Kvzap(wl.d_model, wl.hidden, H, D, L, max_tokens=B, trusted_producers=True)
    weights = []
    for l in range(L):
        wts = synth.surrogate_weights(wl, l, "cuda")
        weights.append(wts)
        ctx.set_weights(l, *wts)
    n_lists = B * L * H
    n_pool = n_lists + 64                             # every list needs at most one page in 4 evictions
    K_pool = torch.zeros(n_pool, P, D, dtype=torch.bfloat16, device="cuda")
    V_pool = torch.zeros_like(K_pool)
    cache = binding.kvzap_cache_create(ctx.handle, B, w, P, K_pool, V_pool, 4)
    rng = np.random.default_rng(5)
    sample_lists = [(int(rng.integers(B)), int(rng.integers(L)), int(rng.integers(H))) for _ in range(48)]
    sample_lists += [(0, 0, 0), (B - 1, L - 1, H - 1), (31, 3, 7), (32, 3, 0), (127, 0, 0)]
    sample_lists = sorted(set(sample_lists))
    check_steps = {0: [0, L - 1], w: [17], n_steps - 1: [5]}
    Xs, Ks, Vs = [], [], []
    for step in range(n_steps):
        Xs.append(synth.hidden_states(L * B, wl.d_model, 9000 + step, "cuda").view(L, B, wl.d_model))
        Kn, Vn = synth.keys_values(L * B, H, D, 9500 + step, "cuda")
        Ks.append(Kn.view(L, B, H, D))
        Vs.append(Vn.view(L, B, H, D))
    scores_all = torch.empty(n_steps, L, B, H, dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    for step in range(n_steps):                       # no synchronisation between steps
        binding.kvzap_decode_step(ctx.handle, cache, 0, L, Xs[step], Ks[step], Vs[step], wl.tau, scores_all[step])
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    s_all = scores_all.cpu().numpy()
    for step, layers in check_steps.items():
        for l in layers:
            want = oracle.score(synth.bits(Xs[step][l]), parity.weights_to_oracle(tuple(t.cpu() for t in weights[l])))
            assert np.abs(s_all[step, l] - want).max() <= parity.SCORE_ATOL
    dec = oracle.DecodeOracle(B, L, H, D, w)          # only the sampled lists are fed
    idx_b = torch.tensor([x[0] for x in sample_lists], device="cuda")
    idx_l = torch.tensor([x[1] for x in sample_lists], device="cuda")
    idx_h = torch.tensor([x[2] for x in sample_lists], device="cuda")
    for step in range(n_steps):
        Kb = synth.bits(Ks[step][idx_l, idx_b, idx_h])         # [n_sample, D]
        Vb = synth.bits(Vs[step][idx_l, idx_b, idx_h])
        for i, (b, l, h) in enumerate(sample_lists):
            win = dec.window[b][l][h]
            win.append((step, np.float32(s_all[step, l, b, h]), Kb[i].copy(), Vb[i].copy()))
            if len(win) > w:
                p_, s_, kr, vr = win.popleft()
                if s_ >= np.float32(wl.tau):
                    dec.prefix[b][l][h].append((p_, kr, vr))
    lengths = torch.zeros(B, L, H, dtype=torch.int32, device="cuda")
    binding.kvzap_cache_lengths(ctx.handle, cache, lengths)
    ln = lengths.cpu().numpy()
    assert (ln >= w).all() and (ln <= n_steps).all()
    # every list: rows held = window + tokens that left it with a score >= tau (from the GPU's own scores)
    kept_exit = (s_all[:n_steps - w] >= np.float32(wl.tau)).sum(axis=0)          # [L, B, H]
    np.testing.assert_array_equal(ln, w + kept_exit.transpose(1, 0, 2))
    K_out = torch.zeros(n_steps, D, dtype=torch.bfloat16, device="cuda")
    V_out = torch.zeros_like(K_out)
    n_rows = torch.zeros(1, dtype=torch.int32, device="cuda")
    for (b, l, h) in sample_lists:
        binding.kvzap_cache_export(ctx.handle, cache, b, l, h, K_out, V_out, n_rows)
        torch.cuda.synchronize()
        n = int(n_rows.item())
        _pos, Kd, Vd = dec.logical(b, l, h)
        assert n == len(Kd) == ln[b, l, h]
        np.testing.assert_array_equal(synth.bits(K_out)[:n], Kd)
        np.testing.assert_array_equal(synth.bits(V_out)[:n], Vd)
    binding.kvzap_cache_destroy(cache)
    ctx.close()
