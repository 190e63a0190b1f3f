"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, prefill.

Sizes span several 128-token tiles with ragged tails; edge cases cover empty
and one-token inputs, T < w, w = 0, w >= T, tau = +-inf, NaN scores, packed
batches with unequal (and empty) sequences, fewer than 8 heads.
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


def _make_ctx(binding, d_model, hidden, H, D, max_tokens, max_seqs=1, n_layers=1):
    return binding.Kvzap(d_model, hidden, H, D, n_layers, max_tokens, max_seqs)


def _weights(d_model, hidden, H, seed, bias_sigma=0.3):
    if hidden == 0:
        return synth.linear_weights(d_model, H, seed, "cpu", bias_sigma)
    return synth.mlp_weights(d_model, hidden, H, seed, "cpu", bias_sigma)


@pytest.mark.parametrize("T", [1, 2, 127, 128, 129, 255, 1000, 4097])
def test_linear_scores_match_oracle(binding, oracle, T):
    d_model, H = 4096 if T <= 255 else 1024, 8
    ctx = _make_ctx(binding, d_model, 0, H, 128, max_tokens=8192)
    weights = _weights(d_model, 0, H, seed=100 + T)
    ctx.set_weights(0, *[parity.dev(w) for w in weights])
    X = synth.hidden_states(T, d_model, seed=T)
    scores = ctx.score(0, parity.dev(X))
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    parity.check_scores(oracle, scores, X, weights)
    ctx.close()


@pytest.mark.parametrize("d_model,hidden,T", [(256, 64, 300), (512, 128, 129), (256, 256, 257), (256, 512, 520),
                                              (256, 640, 200), (128, 1024, 131), (4096, 512, 260), (5120, 640, 130),
                                              (1024, 512, 700), (512, 384, 1000), (2048, 1024, 300),
                                              # 47 and 71 tiles: two CTAs per tile, one per half of the hidden units
                                              (256, 128, 6000), (512, 256, 9000),
                                              # 12 tiles of an MLP whose width allows eight CTAs per tile
                                              (512, 256, 1500)])
def test_mlp_scores_match_oracle(binding, oracle, d_model, hidden, T):
    H = 8
    ctx = _make_ctx(binding, d_model, hidden, H, 128, max_tokens=max(1024, T))
    weights = _weights(d_model, hidden, H, seed=hidden + T)
    ctx.set_weights(0, *[parity.dev(w) for w in weights])
    X = synth.hidden_states(T, d_model, seed=7 * T)
    scores = ctx.score(0, parity.dev(X))
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    parity.check_scores(oracle, scores, X, weights)
    ctx.close()


@pytest.mark.parametrize("H", [1, 3, 5])
@pytest.mark.parametrize("hidden", [0, 128])
def test_fewer_than_eight_heads(binding, oracle, H, hidden):
    d_model, T, D = 256, 333, 64
    ctx = _make_ctx(binding, d_model, hidden, H, D, max_tokens=512)
    weights = _weights(d_model, hidden, H, seed=H * 10 + hidden)
    ctx.set_weights(0, *[parity.dev(w) for w in weights])
    X = synth.hidden_states(T, d_model, seed=3)
    K, V = synth.keys_values(H, T, D, seed=4)
    K_out, V_out = parity.dev(parity.poison_like(K)), parity.dev(parity.poison_like(V))
    scores = torch.empty(T, H, dtype=torch.float32, device="cuda")
    _, _, lengths = ctx.prefill_fused(0, parity.dev(X), parity.dev(K), parity.dev(V), 0.1, 16,
                                      K_out=K_out, V_out=V_out, scores_out=scores)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    want, _ = parity.check_scores(oracle, scores, X, weights)
    s = scores.cpu().numpy()
    parity.check_mask_band(oracle, s, want, 0.1, 16, None)
    parity.check_compaction(oracle, K, V, s, 0.1, 16, None, K_out, V_out, lengths)
    ctx.close()


def _run_fused(binding, oracle, d_model, hidden, H, D, seq_lens, tau, w, seed, token_scale_sigma=0.0):
    T = int(sum(seq_lens))
    B = len(seq_lens)
    ctx = _make_ctx(binding, d_model, hidden, H, D, max_tokens=max(T, 1), max_seqs=B)
    weights = _weights(d_model, hidden, H, seed=seed)
    ctx.set_weights(0, *[parity.dev(w_) for w_ in weights])
    X = synth.hidden_states(T, d_model, seed=seed + 1, token_scale_sigma=token_scale_sigma)
    K, V = synth.keys_values(H, T, D, seed=seed + 2)
    cu = synth.cu_seqlens(seq_lens)
    cu_dev = torch.from_numpy(cu).cuda() if B > 1 else None
    K_out, V_out = parity.dev(parity.poison_like(K)), parity.dev(parity.poison_like(V))
    scores = torch.full((T, H), float("nan"), dtype=torch.float32, device="cuda")
    _, _, lengths = ctx.prefill_fused(0, parity.dev(X), parity.dev(K), parity.dev(V), tau, w, cu_seqlens=cu_dev,
                                      K_out=K_out, V_out=V_out, scores_out=scores)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    want, err = parity.check_scores(oracle, scores, X, weights)
    s = scores.cpu().numpy()
    cu_arg = cu if B > 1 else None
    parity.check_mask_band(oracle, s, want, tau, w, cu_arg)
    keep, len_ref = parity.check_compaction(oracle, K, V, s, tau, w, cu_arg, K_out, V_out, lengths)
    # the same result without asking for the scores
    K2, V2 = parity.dev(parity.poison_like(K)), parity.dev(parity.poison_like(V))
    _, _, len2 = ctx.prefill_fused(0, parity.dev(X), parity.dev(K), parity.dev(V), tau, w, cu_seqlens=cu_dev,
                                   K_out=K2, V_out=V2)
    torch.cuda.synchronize()
    assert torch.equal(len2, lengths) and torch.equal(K2.view(torch.int16), K_out.view(torch.int16))
    assert torch.equal(V2.view(torch.int16), V_out.view(torch.int16))
    # and through the two-call route (score, then prune) on the same scores
    K3, V3 = parity.dev(parity.poison_like(K)), parity.dev(parity.poison_like(V))
    _, _, len3 = ctx.prune_prefill(parity.dev(K), parity.dev(V), scores, tau, w, cu_seqlens=cu_dev, K_out=K3, V_out=V3)
    torch.cuda.synchronize()
    assert torch.equal(len3, lengths) and torch.equal(K3.view(torch.int16), K_out.view(torch.int16))
    assert torch.equal(V3.view(torch.int16), V_out.view(torch.int16))
    ctx.close()
    return keep, len_ref


@pytest.mark.parametrize("T,w,tau", [(1, 128, 0.43), (2, 0, 0.0), (100, 128, 0.43), (128, 128, 0.43), (129, 128, 0.43),
                                     (700, 128, 0.43), (700, 0, 0.43), (700, 512, -0.5), (700, 1000, 0.43),
                                     (1300, 128, float("inf")), (1300, 128, float("-inf")), (4097, 128, 0.84),
                                     # 47, 63 and 64 tiles: scoring and compaction in one launch with several CTAs per SM;
                                     # 65 tiles: the first length that takes two launches again
                                     (6000, 128, 0.43), (8001, 64, 0.0), (8192, 128, 0.43), (8200, 128, 0.43)])
def test_fused_linear_single_sequence(binding, oracle, T, w, tau):
    keep, lengths = _run_fused(binding, oracle, 512, 0, 8, 128, [T], tau, w, seed=T + w)
    assert (lengths >= min(T, w)).all()
    if tau == float("inf"):
        assert (lengths == min(T, w)).all()
    if tau == float("-inf") or w >= T:
        assert (lengths == T).all()


@pytest.mark.parametrize("hidden,T", [(64, 300), (512, 600), (640, 257), (128, 7000)])
def test_fused_mlp_single_sequence(binding, oracle, hidden, T):
    _run_fused(binding, oracle, 256, hidden, 8, 128, [T], 0.2, 128, seed=hidden)


@pytest.mark.parametrize("seq_lens", [[5, 40, 1, 0, 17], [128, 128], [300, 77, 0, 0, 900, 1], [1, 1, 1, 1]])
@pytest.mark.parametrize("hidden", [0, 128])
def test_fused_packed_batch_windows_are_per_sequence(binding, oracle, seq_lens, hidden):
    keep, lengths = _run_fused(binding, oracle, 256, hidden, 8, 64, seq_lens, 0.43, 8, seed=len(seq_lens),
                               token_scale_sigma=0.5)
    for b, n in enumerate(seq_lens):
        assert (lengths[b] >= min(n, 8)).all() and (lengths[b] <= n).all()


def test_prune_with_nan_inf_scores_and_other_head_dims(binding, oracle):
    for D in (8, 64, 256):
        H, T, w, tau = 8, 777, 16, 0.25
        rng = np.random.default_rng(D)
        s = rng.standard_normal((T, H)).astype(np.float32)
        s[5, 0] = np.nan
        s[6, 1] = np.inf
        s[7, 2] = -np.inf
        s[8, 3] = np.float32(tau)                   # tie is kept
        s[T - 3, 4] = np.nan                        # NaN inside the window is kept
        K, V = synth.keys_values(H, T, D, seed=D)
        ctx = _make_ctx(binding, 256, 0, H, D, max_tokens=T)
        K_out, V_out = parity.dev(parity.poison_like(K)), parity.dev(parity.poison_like(V))
        _, _, lengths = ctx.prune_prefill(parity.dev(K), parity.dev(V), torch.from_numpy(s).cuda(), tau, w,
                                          K_out=K_out, V_out=V_out)
        torch.cuda.synchronize()
        keep, _ = parity.check_compaction(oracle, K, V, s, tau, w, None, K_out, V_out, lengths)
        assert keep[0, 5] == 0 and keep[1, 6] == 1 and keep[2, 7] == 0 and keep[3, 8] == 1 and keep[4, T - 3] == 1
        ctx.close()


def test_empty_input_and_argument_errors(binding):
    ctx = _make_ctx(binding, 256, 0, 8, 128, max_tokens=256, max_seqs=2)
    W, b = synth.linear_weights(256, 8, 1)
    K = torch.empty(8, 0, 128, dtype=torch.bfloat16, device="cuda")
    lengths = torch.full((1, 8), -7, dtype=torch.int32, device="cuda")
    # scoring a layer that has no weights yet is a state error
    with pytest.raises(binding.KvzapError) as ei:
        ctx.score(0, torch.zeros(4, 256, dtype=torch.bfloat16, device="cuda"))
    assert ei.value.status == 6
    ctx.set_weights(0, parity.dev(W), parity.dev(b))
    ctx.prune_prefill(K, K, torch.empty(0, 8, device="cuda"), 0.0, 4, K_out=K, V_out=K, lengths=lengths)
    torch.cuda.synchronize()
    assert (lengths == 0).all()
    assert ctx.score(0, torch.empty(0, 256, dtype=torch.bfloat16, device="cuda")).shape == (0, 8)
    with pytest.raises(binding.KvzapError) as ei:      # more tokens than the context was sized for
        ctx.score(0, torch.zeros(257, 256, dtype=torch.bfloat16, device="cuda"))
    assert ei.value.status == 1
    K1 = torch.zeros(8, 16, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.KvzapError) as ei:      # negative window
        ctx.prune_prefill(K1, K1, torch.zeros(16, 8, device="cuda"), 0.0, -1)
    assert ei.value.status == 1
    with pytest.raises(binding.KvzapError):            # layer out of range
        ctx.score(3, torch.zeros(4, 256, dtype=torch.bfloat16, device="cuda"))
    assert ctx.poll_status() == 0
    ctx.close()


def test_larger_tau_keeps_a_subset_on_the_gpu(binding, oracle):
    T, H, D = 2000, 8, 128
    ctx = _make_ctx(binding, 512, 0, H, D, max_tokens=T)
    weights = _weights(512, 0, H, seed=9, bias_sigma=0.0)
    ctx.set_weights(0, *[parity.dev(w) for w in weights])
    X = parity.dev(synth.hidden_states(T, 512, seed=10))
    K, V = synth.keys_values(H, T, D, seed=11)
    # tag every K row with its position so that the kept positions can be read back
    Kb = synth.bits(K).copy()
    Kb[:, :, 0] = np.arange(T, dtype=np.uint16)[None, :]
    Kd, Vd = synth.from_bits(Kb, "cuda"), parity.dev(V)
    prev = None
    for tau in [-1.0, 0.0, 0.43, 0.84]:
        K_out, _, lengths = ctx.prefill_fused(0, X, Kd, Vd, tau, 128)
        torch.cuda.synchronize()
        Ko, ln = synth.bits(K_out), lengths.cpu().numpy()
        kept = [set(Ko[h, :ln[0, h], 0].tolist()) for h in range(H)]
        for h in range(H):
            assert set(range(T - 128, T)) <= kept[h]                    # the window is always kept
            pos = Ko[h, :ln[0, h], 0].astype(np.int64)
            assert np.all(np.diff(pos) > 0)                             # token order preserved
            if prev is not None:
                assert kept[h] <= prev[h]
        prev = kept
    ctx.close()


@pytest.mark.parametrize("seq_lens,H,D,P", [
    ([131072 + 77], 8, 128, 0),                         # more blocks than CTAs: several blocks per CTA
    ([40000, 1, 0, 50011, 129, 30000], 8, 64, 0),       # sequences that start inside a CTA's run of blocks
    ([131072 + 77], 8, 128, 16),                        # the same, paged: the last CTA to arrive assigns the pages
    ([40000, 1, 0, 50011, 129, 30000], 5, 64, 16),
    ([2600000, 17], 2, 8, 0),                           # more than 32 blocks per CTA: mask words re-read from memory
    ([2600000, 17], 2, 8, 5),
])
def test_prune_prefill_one_launch_many_blocks_per_cta(binding, oracle, seq_lens, H, D, P):
    """kvzap_prune_prefill / _paged on given scores at sizes where a CTA of the one-launch kernel owns
    several (and more than 32) blocks and sequences begin in the middle of a CTA's run; lengths, rows,
    page tables and untouched memory bit for bit against the oracle's mask and ordered gather."""
    T, B, tau, w = int(sum(seq_lens)), len(seq_lens), 0.43, 128
    ctx = binding.Kvzap(256, 0, H, D, 1, T, max_seqs=B, trusted_producers=True)
    g = torch.Generator(device="cuda").manual_seed(T % 1000 + H)
    scores = torch.randn(T, H, generator=g, device="cuda")
    K, V = synth.keys_values(H, T, D, seed=3, device="cuda")
    cu = synth.cu_seqlens(seq_lens)
    cu_dev = torch.from_numpy(cu).cuda() if B > 1 else None
    cu_arg = cu if B > 1 else None
    s_np = scores.cpu().numpy()
    for rep in range(2):                                # twice in a row: the second launch starts under the first
        if P == 0:
            K_out, V_out = parity.poison_like(K), parity.poison_like(V)
            lengths = torch.full((B, H), -1, dtype=torch.int32, device="cuda")
            binding.kvzap_prune_prefill(ctx.handle, K, V, scores, cu_dev, B, tau, w, K_out, V_out, lengths)
        else:
            n_pool, max_pages, first_page = H * (T // P + B + 1) // 2 + 7, max(seq_lens) // P + 2, 3
            K_pool = torch.full((n_pool, P, D), -5.0, dtype=torch.bfloat16, device="cuda")
            V_pool = torch.full((n_pool, P, D), -5.0, dtype=torch.bfloat16, device="cuda")
            table = torch.full((B * H, max_pages), -1, dtype=torch.int32, device="cuda")
            lengths = torch.zeros(B, H, dtype=torch.int32, device="cuda")
            used = torch.zeros(1, dtype=torch.int32, device="cuda")
            binding.kvzap_prune_prefill_paged(ctx.handle, K, V, scores, cu_dev, B, tau, w, K_pool, V_pool, P, first_page,
                                              table, lengths, used)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    if P == 0:
        parity.check_compaction(oracle, K.cpu(), V.cpu(), s_np, tau, w, cu_arg, K_out.cpu(), V_out.cpu(), lengths)
    else:
        keep = oracle.keep_mask(s_np, tau, w, cu_arg)
        fill = int(synth.bits(torch.tensor([-5.0], dtype=torch.bfloat16))[0])
        Kp, Vp, tab, ln, n_used = oracle.compact_paged(synth.bits(K), synth.bits(V), keep, P, n_pool, max_pages,
                                                       cu_seqlens=cu_arg, first_page=first_page, fill=fill)
        np.testing.assert_array_equal(lengths.cpu().numpy(), ln)
        assert int(used.item()) == n_used
        np.testing.assert_array_equal(table.cpu().numpy(), tab)
        np.testing.assert_array_equal(synth.bits(K_pool), Kp)
        np.testing.assert_array_equal(synth.bits(V_pool), Vp)
    ctx.close()
