"""GPU parity for attention over a pruned cache of 8-bit rows, against the CPU oracle.

Rows are E4M3 codes followed by a 16-byte trailer that starts with the row's fp32 scale (Related work,
"Quantization": quantisation and pruning of the cache compose).  The pruning calls move such rows as opaque
bytes, so the cache is driven exactly as in the bf16 tests (the decode oracle follows the GPU's scores) and the
oracle's copy of a list, unpacked into codes and scales, goes through the oracle's 8-bit attention.

Tolerance: codes widen exactly, the logits accumulate in fp32, probabilities times the V scale are rounded to
bf16 (relative 2^-9) before the second product and the output is rounded to bf16 once; ATTN_ATOL = 2e-2
(outputs of order one) covers both with room.
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


def _weights(d_model, hidden, H, seed):
    if hidden == 0:
        return synth.linear_weights(d_model, H, seed, "cpu", 0.3)
    return synth.mlp_weights(d_model, hidden, H, seed, "cpu", 0.3)


def _poisoned_pool(n_pool, P, Dr):
    """NaN bit patterns as bf16 words: as bytes, 0x7f is the NaN code and the scale is a NaN too."""
    return torch.full((n_pool, P, Dr), float("nan"), dtype=torch.bfloat16, device="cuda")


def _want(oracle, qbits, Krows, Vrows, D, scale):
    K8, ks = synth.unpack_rows_e4m3(Krows, D)
    V8, vs = synth.unpack_rows_e4m3(Vrows, D)
    return oracle.attention_fp8(qbits, K8, ks, V8, vs, scale)


def _check(binding, oracle, ctx, cache, dec, L, B, H, G, D, seed):
    Q = synth.hidden_states(L * B * H * G, D, seed=seed).view(L, B, H * G, D)
    O = torch.full((L, B, H * G, D), 7.0, dtype=torch.bfloat16, device="cuda")
    scale = 1.0 / np.sqrt(D)
    binding.kvzap_decode_attention_fp8(ctx.handle, cache, 0, L, parity.dev(Q), scale, O)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    got = O.float().cpu().numpy()
    assert np.isfinite(got).all()
    Qb = synth.bits(Q)
    worst = 0.0
    for l in range(L):
        for b in range(B):
            for h in range(H):
                _pos, Kd, Vd = dec.logical(b, l, h)
                if len(Kd) == 0:
                    want = np.zeros((G, D), dtype=np.float32)
                else:
                    want = _want(oracle, Qb[l, b, h * G:(h + 1) * G], Kd, Vd, D, scale)
                worst = max(worst, float(np.abs(got[l, b, h * G:(h + 1) * G] - want).max()))
    assert worst <= ATTN_ATOL, worst
    return worst


@pytest.mark.parametrize("hidden,w,P,B,L,D,G", [
    (128, 16, 16, 3, 2, 128, 4),
    (0, 32, 16, 2, 1, 64, 4),
    (64, 0, 16, 2, 1, 128, 8),        # no window: a new token is decided at once
    (128, 16, 32, 5, 1, 128, 1),      # two tiles per page, one query head per KV head
])
def test_attention_fp8_after_decode_steps(binding, oracle, hidden, w, P, B, L, D, G):
    d_model, H, tau, n_steps = 256, 8, -0.2, 100
    Dr = (D + synth.E4M3_ROW_TRAILER) // 2            # row width in bf16 units, as the context sees it
    ctx = binding.Kvzap(d_model, hidden, H, Dr, L, max_tokens=128, max_seqs=1)
    for l in range(L):
        ctx.set_weights(l, *[parity.dev(x) for x in _weights(d_model, hidden, H, seed=70 + l)])
    max_pages = n_steps // P + 2
    n_pool = B * L * H * max_pages
    K_pool, V_pool = _poisoned_pool(n_pool, P, Dr), _poisoned_pool(n_pool, P, Dr)
    cache = binding.kvzap_cache_create(ctx.handle, B, w, P, K_pool, V_pool, max_pages)
    dec = oracle.DecodeOracle(B, L, H, Dr, w)
    for step in range(n_steps):
        X = synth.hidden_states(L * B, d_model, seed=3000 + step).view(L, B, d_model)
        Kf, Vf = synth.keys_values(L * B, H, D, seed=4000 + step)
        # rows of very different magnitudes, so that a scale applied to the wrong row shows (V stays of order one:
        # the tolerance is an absolute one on outputs that are rounded to bf16)
        mag = torch.from_numpy(np.random.default_rng(step).uniform(0.05, 8.0, size=(L * B, H, 1)).astype(np.float32))
        K_new = synth.pack_rows_e4m3(Kf.float() * mag).view(L, B, H, Dr)
        V_new = synth.pack_rows_e4m3(Vf.float() * (mag.flip(0) / 8.0)).view(L, B, H, Dr)
        scores = torch.empty(L, B, H, dtype=torch.float32, device="cuda")
        binding.kvzap_decode_step(ctx.handle, cache, 0, L, parity.dev(X), parity.dev(K_new), parity.dev(V_new), tau, scores)
        torch.cuda.synchronize()
        s = scores.cpu().numpy()
        for l in range(L):
            Kb, Vb = synth.bits(K_new[l]), synth.bits(V_new[l])
            for b in range(B):
                dec.append(b, l, s[l, b], Kb[b], Vb[b], tau)
        if step in (0, 4, max(w - 1, 1), w + 1, 57, n_steps - 1):
            _check(binding, oracle, ctx, cache, dec, L, B, H, G, D, seed=9000 + step)
    binding.kvzap_cache_destroy(cache)
    ctx.close()


@pytest.mark.parametrize("B,lo,hi", [(128, 1000, 8000), (300, 200, 2000)])
def test_attention_fp8_at_bench_size_sampled_lists(binding, oracle, B, lo, hi):
    """128 sequences x 8 KV heads with lists of 1k..8k pruned rows plus a full window of 128 (lists cut into
    parts), and 300 sequences (one CTA per list): sampled lists against the oracle."""
    d_model, H, D, P, w, G = 256, 8, 128, 16, 128, 4
    Dr = (D + synth.E4M3_ROW_TRAILER) // 2
    ctx = binding.Kvzap(d_model, 0, H, Dr, 1, max_tokens=B)
    W, bias = synth.linear_weights(d_model, H, 3)
    ctx.set_weights(0, parity.dev(W), parity.dev(bias))
    n_lists = B * H
    rng = np.random.default_rng(99)
    prefix = rng.integers(lo, hi + 1, size=n_lists).astype(np.int32)
    prefix[:4] = [1, 15, 16, 17]
    pages_of = (prefix + P - 1) // P
    first = np.concatenate([[0], np.cumsum(pages_of)[:-1]]).astype(np.int64)
    n_pool, max_pages = int(pages_of.sum()), int(pages_of.max())
    Kf, Vf = synth.keys_values(1, n_pool * P, D, seed=123, device="cuda")
    mag = torch.from_numpy(rng.uniform(0.05, 8.0, size=(n_pool * P, 1)).astype(np.float32)).cuda()
    K_pool = synth.pack_rows_e4m3(Kf[0].float() * mag).view(n_pool, P, Dr)
    V_pool = synth.pack_rows_e4m3(Vf[0].float() * (mag.flip(0) / 8.0)).view(n_pool, P, Dr)
    last_fill = prefix - (pages_of - 1) * P
    for li in range(0, n_lists, 37):       # rows past a list's end inside its last page must not matter
        pg = int(first[li] + pages_of[li] - 1)
        K_pool[pg, int(last_fill[li]):] = float("nan")
        V_pool[pg, int(last_fill[li]):] = float("nan")
    table = torch.from_numpy((first[:, None] + np.arange(max_pages)[None, :]).astype(np.int32)).cuda()
    cache = binding.kvzap_cache_create(ctx.handle, B, w, P, K_pool, V_pool, max_pages)
    binding.kvzap_cache_import(ctx.handle, cache, torch.from_numpy(prefix).cuda(), table, n_pool)
    n_steps = w + 3
    new_rows = []
    for step in range(n_steps):
        X = parity.dev(synth.hidden_states(B, d_model, seed=600 + step)).view(1, B, d_model)
        Kn, Vn = synth.keys_values(B, H, D, seed=700 + step)
        Kn, Vn = synth.pack_rows_e4m3(Kn.float() * 3.0), synth.pack_rows_e4m3(Vn.float() * 0.25)
        new_rows.append((synth.bits(Kn), synth.bits(Vn)))
        binding.kvzap_decode_step(ctx.handle, cache, 0, 1, X, parity.dev(Kn).view(1, B, H, Dr),
                                  parity.dev(Vn).view(1, B, H, Dr), float("inf"), None)    # nothing joins the prefix
    Q = synth.hidden_states(B * H * G, D, seed=8).view(1, B, H * G, D)
    O = torch.zeros(1, B, H * G, D, dtype=torch.bfloat16, device="cuda")
    scale = 1.0 / np.sqrt(D)
    binding.kvzap_decode_attention_fp8(ctx.handle, cache, 0, 1, parity.dev(Q), scale, O)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    got = O.float().cpu().numpy()[0]
    assert np.isfinite(got).all()
    Qb = synth.bits(Q)[0]
    Kp_bits, Vp_bits = synth.bits(K_pool.cpu()).reshape(-1, Dr), synth.bits(V_pool.cpu()).reshape(-1, Dr)
    sample = sorted(set([0, 1, 2, 3, 37, 74, n_lists - 1] + rng.integers(0, n_lists, 20).tolist()))
    for li in sample:
        b, h = li // H, li % H
        r0 = int(first[li]) * P
        Kd = np.concatenate([Kp_bits[r0:r0 + int(prefix[li])]] + [new_rows[s][0][b, h][None] for s in range(n_steps - w, n_steps)])
        Vd = np.concatenate([Vp_bits[r0:r0 + int(prefix[li])]] + [new_rows[s][1][b, h][None] for s in range(n_steps - w, n_steps)])
        want = _want(oracle, Qb[b, h * G:(h + 1) * G], Kd, Vd, D, scale)
        assert np.abs(got[b, h * G:(h + 1) * G] - want).max() <= ATTN_ATOL, li
    binding.kvzap_cache_destroy(cache)
    ctx.close()


def test_attention_fp8_argument_checks(binding):
    d_model, H, P, w = 256, 8, 16, 16
    ctx = binding.Kvzap(d_model, 0, H, 72, 1, max_tokens=16)
    pool = torch.zeros(H * 4, P, 72, dtype=torch.bfloat16, device="cuda")
    cache = binding.kvzap_cache_create(ctx.handle, 1, w, P, pool, pool.clone(), 4)
    Q = torch.zeros(1, 1, 32, 128, dtype=torch.bfloat16, device="cuda")
    O = torch.ones_like(Q)
    binding.kvzap_decode_attention_fp8(ctx.handle, cache, 0, 1, Q, 0.1, O)       # empty lists: zeros
    torch.cuda.synchronize()
    assert float(O.float().abs().max()) == 0.0
    with pytest.raises(binding.KvzapError):
        binding.kvzap_decode_attention(ctx.handle, cache, 0, 1, Q, 0.1, O)        # rows of 72 bf16 values: not a bf16 cache
    binding.kvzap_cache_destroy(cache)
    ctx.close()
    ctx = binding.Kvzap(d_model, 0, H, 128, 1, max_tokens=16)                      # 256-byte rows: neither 64 nor 128 codes
    pool = torch.zeros(H * 4, P, 128, dtype=torch.bfloat16, device="cuda")
    cache = binding.kvzap_cache_create(ctx.handle, 1, w, P, pool, pool.clone(), 4)
    with pytest.raises(binding.KvzapError):
        binding.kvzap_decode_attention_fp8(ctx.handle, cache, 0, 1, Q, 0.1, O)
    binding.kvzap_cache_destroy(cache)
    ctx.close()
