"""GPU parity for write-side pruning: K and V in the projection's layout [T, H, D].

Same comparison rules as the head-major calls (tests/parity.py): scores within the
tolerance, mask equal outside the tolerance band, then lengths, rows, pages and page
tables bit for bit against the oracle's write-side compaction run on the GPU's own
scores.  The head-major call on the transposed input must give the same bits too.
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


def _inputs(T, d_model, H, D, seed):
    X = synth.hidden_states(T, d_model, seed=seed)
    K, V = synth.keys_values(H, T, D, seed=seed + 1)             # [H, T, D]
    K_proj = K.transpose(0, 1).contiguous()                      # [T, H, D]: a pure relabelling of the draws
    V_proj = V.transpose(0, 1).contiguous()
    return X, K, V, K_proj, V_proj


@pytest.mark.parametrize("seq_lens,hidden,H,D,w,tau", [
    ([700], 0, 8, 128, 16, 0.3),            # several tiles and a ragged tail
    ([1], 0, 8, 128, 4, 0.0),               # T < w
    ([129], 128, 8, 64, 0, 0.2),            # no window
    ([37, 64, 5, 0, 300], 128, 8, 128, 16, 0.3),
    ([1000, 24, 333], 64, 5, 32, 128, -0.1),    # fewer heads, short rows, a sequence shorter than w
    ([4096], 256, 8, 128, 128, 0.43),
])
def test_write_side_dense_matches_oracle(binding, oracle, seq_lens, hidden, H, D, w, tau):
    d_model = 256 if hidden != 256 else 2048
    T, B = int(sum(seq_lens)), len(seq_lens)
    ctx = binding.Kvzap(d_model, hidden, H, D, 1, T, max_seqs=B)
    weights = _weights(d_model, hidden, H, seed=T + hidden)
    ctx.set_weights(0, *[parity.dev(x) for x in weights])
    X, K, V, K_proj, V_proj = _inputs(T, d_model, H, D, seed=T)
    cu = synth.cu_seqlens(seq_lens)
    cu_dev = torch.from_numpy(cu).cuda() if B > 1 else None
    cu_arg = cu if B > 1 else None
    K_out = parity.poison_like(torch.empty(H, T, D, dtype=torch.bfloat16, device="cuda"))
    V_out = parity.poison_like(K_out)
    lengths = torch.full((B, H), -7, dtype=torch.int32, device="cuda")
    scores = torch.empty(T, H, dtype=torch.float32, device="cuda")
    binding.kvzap_prefill_write(ctx.handle, 0, parity.dev(X), parity.dev(K_proj), parity.dev(V_proj), cu_dev, B, tau, w,
                                K_out, V_out, lengths, scores)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    want, _ = parity.check_scores(oracle, scores, X, weights)
    s = scores.cpu().numpy()
    keep = parity.check_mask_band(oracle, s, want, tau, w, cu_arg)
    K_ref, V_ref, len_ref = oracle.compact_write(synth.bits(K_proj), synth.bits(V_proj), keep, cu_arg, fill=parity.POISON)
    np.testing.assert_array_equal(lengths.cpu().numpy(), len_ref)
    np.testing.assert_array_equal(synth.bits(K_out), K_ref)          # the poison past lengths included
    np.testing.assert_array_equal(synth.bits(V_out), V_ref)
    # the head-major call on the transposed input gives the same bits
    K2, V2 = parity.poison_like(K_out), parity.poison_like(K_out)
    len2 = torch.zeros_like(lengths)
    binding.kvzap_prefill_fused(ctx.handle, 0, parity.dev(X), parity.dev(K), parity.dev(V), cu_dev, B, tau, w, K2, V2, len2)
    torch.cuda.synchronize()
    assert torch.equal(len2, lengths)
    assert torch.equal(K2.view(torch.int16), K_out.view(torch.int16))
    assert torch.equal(V2.view(torch.int16), V_out.view(torch.int16))
    ctx.close()


@pytest.mark.parametrize("seq_lens,hidden,P", [([700], 0, 16), ([37, 64, 5, 0, 300], 128, 16), ([1000, 24], 0, 7)])
def test_write_side_paged_matches_oracle(binding, oracle, seq_lens, hidden, P):
    d_model, H, D, tau, w = 256, 8, 64, 0.3, 16
    T, B = int(sum(seq_lens)), len(seq_lens)
    ctx = binding.Kvzap(d_model, hidden, H, D, 1, T, max_seqs=B)
    weights = _weights(d_model, hidden, H, seed=B + hidden)
    ctx.set_weights(0, *[parity.dev(x) for x in weights])
    X, K, V, K_proj, V_proj = _inputs(T, d_model, H, D, seed=11)
    cu = synth.cu_seqlens(seq_lens)
    cu_dev = torch.from_numpy(cu).cuda() if B > 1 else None
    cu_arg = cu if B > 1 else None
    n_pool, max_pages, first_page = H * (T // P + B + 1) + 5, max(seq_lens) // P + 2, 3
    pool = lambda: torch.full((n_pool, P, D), -5.0, dtype=torch.bfloat16, device="cuda")
    K_pool, V_pool = pool(), pool()
    table = torch.full((B * H, max_pages), -1, dtype=torch.int32, device="cuda")
    lengths = torch.zeros(B, H, dtype=torch.int32, device="cuda")
    used = torch.zeros(1, dtype=torch.int32, device="cuda")
    scores = torch.empty(T, H, dtype=torch.float32, device="cuda")
    binding.kvzap_prefill_write_paged(ctx.handle, 0, parity.dev(X), parity.dev(K_proj), parity.dev(V_proj), cu_dev, B, tau,
                                      w, K_pool, V_pool, P, first_page, table, lengths, used, scores)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    want, _ = parity.check_scores(oracle, scores, X, weights)
    s = scores.cpu().numpy()
    keep = parity.check_mask_band(oracle, s, want, tau, w, cu_arg)
    fill = int(synth.bits(torch.tensor([-5.0], dtype=torch.bfloat16))[0])
    Kp, Vp, tab, ln, n_used = oracle.compact_write_paged(synth.bits(K_proj), synth.bits(V_proj), keep, P, n_pool, max_pages,
                                                         cu_seqlens=cu_arg, first_page=first_page, fill=fill)
    np.testing.assert_array_equal(lengths.cpu().numpy(), ln)
    assert int(used.item()) == n_used
    np.testing.assert_array_equal(table.cpu().numpy(), tab)
    np.testing.assert_array_equal(synth.bits(K_pool), Kp)
    np.testing.assert_array_equal(synth.bits(V_pool), Vp)
    ctx.close()


def test_write_side_empty_input_and_argument_errors(binding):
    ctx = binding.Kvzap(256, 0, 8, 128, 1, 1024)
    ctx.set_weights(0, *[parity.dev(x) for x in _weights(256, 0, 8, 1)])
    lengths = torch.full((1, 8), 9, dtype=torch.int32, device="cuda")
    empty = torch.empty(0, 8, 128, dtype=torch.bfloat16, device="cuda")
    binding.kvzap_prefill_write(ctx.handle, 0, torch.empty(0, 256, dtype=torch.bfloat16, device="cuda"), empty, empty,
                                None, 1, 0.0, 4, empty, empty, lengths)
    torch.cuda.synchronize()
    assert (lengths == 0).all()
    X = synth.hidden_states(64, 256, seed=1).cuda()
    Kp = torch.zeros(64, 8, 128, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(8, 64, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.KvzapError):
        binding.kvzap_prefill_write(ctx.handle, 0, X, Kp, Kp, None, 1, 0.0, -1, out, out, lengths)     # w < 0
    with pytest.raises(binding.KvzapError):
        binding.kvzap_prefill_write(ctx.handle, 3, X, Kp, Kp, None, 1, 0.0, 4, out, out, lengths)      # layer out of range
    ctx.close()


def test_write_side_at_config3_size(binding, oracle):
    """Four sequences of 16k tokens, Linear surrogate, K/V as [T,H,D]: everything checked in full."""
    wl = synth.WORKLOADS["llama31_8b_prefill_4x16k"]
    B, T = wl.batch, wl.seq_len
    n_tokens, H, D, tau = B * T, wl.n_kv_heads, wl.head_dim, wl.tau
    ctx = binding.Kvzap(wl.d_model, wl.hidden, H, D, 1, n_tokens, max_seqs=B)
    weights = synth.surrogate_weights(wl, 2, "cuda")
    ctx.set_weights(0, *weights)
    X = synth.hidden_states(n_tokens, wl.d_model, 77, "cuda", wl.token_scale_sigma)
    K, V = synth.keys_values(H, n_tokens, D, 78, "cuda")
    K_proj, V_proj = K.transpose(0, 1).contiguous(), V.transpose(0, 1).contiguous()
    del K, V
    cu = synth.cu_seqlens([T] * B)
    K_out = parity.poison_like(torch.empty(H, n_tokens, D, dtype=torch.bfloat16, device="cuda"))
    V_out = parity.poison_like(K_out)
    lengths = torch.zeros(B, H, dtype=torch.int32, device="cuda")
    scores = torch.empty(n_tokens, H, dtype=torch.float32, device="cuda")
    binding.kvzap_prefill_write(ctx.handle, 0, X, K_proj, V_proj, torch.from_numpy(cu).cuda(), B, tau, wl.window,
                                K_out, V_out, lengths, scores)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    want, _ = parity.check_scores(oracle, scores, X.cpu(), tuple(w.cpu() if w is not None else None for w in weights))
    s = scores.cpu().numpy()
    keep = parity.check_mask_band(oracle, s, want, tau, wl.window, cu)
    K_ref, V_ref, len_ref = oracle.compact_write(synth.bits(K_proj.cpu()), synth.bits(V_proj.cpu()), keep, cu,
                                                 fill=parity.POISON)
    np.testing.assert_array_equal(lengths.cpu().numpy(), len_ref)
    np.testing.assert_array_equal(synth.bits(K_out.cpu()), K_ref)
    np.testing.assert_array_equal(synth.bits(V_out.cpu()), V_ref)
    assert (len_ref >= wl.window).all()
    ctx.close()
