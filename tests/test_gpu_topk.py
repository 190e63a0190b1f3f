"""GPU parity for fixed-budget (top-k) selection: cut values, lengths and compacted rows against
the oracle, bit for bit (the scores are an input here, so nothing is approximate)."""
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


def _run(binding, oracle, seq_lens, H, D, w, ratio, per_layer, scores):
    T, B = int(sum(seq_lens)), len(seq_lens)
    ctx = binding.Kvzap(256, 0, H, D, 1, max(T, 1), max_seqs=B)
    K, V = synth.keys_values(H, T, D, seed=T + 3)
    cu = synth.cu_seqlens(seq_lens)
    cu_dev = torch.from_numpy(cu).cuda() if B > 1 else None
    cu_arg = cu if B > 1 else None
    K_out = parity.poison_like(torch.empty(H, T, D, dtype=torch.bfloat16, device="cuda"))
    V_out = parity.poison_like(K_out)
    lengths = torch.full((B, H), -3, dtype=torch.int32, device="cuda")
    tau = torch.full((B, H), 123.0, dtype=torch.float32, device="cuda")
    s_dev = torch.from_numpy(scores).cuda()
    binding.kvzap_prune_prefill_topk(ctx.handle, parity.dev(K), parity.dev(V), s_dev, cu_dev, B, ratio, w, per_layer,
                                     K_out, V_out, lengths, tau)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    keep, tau_ref = oracle.topk_mask(scores, ratio, w, per_layer, cu_arg)
    np.testing.assert_array_equal(tau.cpu().numpy(), tau_ref)                 # the same cut values (as numbers)
    K_ref, V_ref, len_ref = oracle.compact(synth.bits(K), synth.bits(V), keep, cu_arg, fill=parity.POISON)
    np.testing.assert_array_equal(lengths.cpu().numpy(), len_ref)
    np.testing.assert_array_equal(synth.bits(K_out), K_ref)
    np.testing.assert_array_equal(synth.bits(V_out), V_ref)
    # without tau_out the result is the same
    K2, V2 = parity.poison_like(K_out), parity.poison_like(K_out)
    len2 = torch.zeros_like(lengths)
    binding.kvzap_prune_prefill_topk(ctx.handle, parity.dev(K), parity.dev(V), s_dev, cu_dev, B, ratio, w, per_layer,
                                     K2, V2, len2)
    torch.cuda.synchronize()
    assert torch.equal(len2, lengths) and torch.equal(K2.view(torch.int16), K_out.view(torch.int16))
    ctx.close()
    return len_ref


@pytest.mark.parametrize("per_layer", [False, True])
@pytest.mark.parametrize("seq_lens,H,w,ratio", [
    ([700], 8, 16, 0.25),
    ([37, 64, 5, 0, 300, 1], 8, 16, 0.4),       # packed batch, empty and tiny sequences, T_b < w
    ([1000], 5, 0, 0.1),                        # no window, fewer heads
    ([513], 8, 128, 1.0),                       # everything
    ([513], 8, 128, 0.0),                       # the window alone
])
def test_topk_random_scores(binding, oracle, seq_lens, H, w, ratio, per_layer):
    rng = np.random.default_rng(sum(seq_lens) + H)
    s = rng.standard_normal((sum(seq_lens), H)).astype(np.float32)
    _run(binding, oracle, seq_lens, H, 64, w, ratio, per_layer, s)


@pytest.mark.parametrize("per_layer", [False, True])
def test_topk_ties_signed_zeros_nan_inf(binding, oracle, per_layer):
    rng = np.random.default_rng(3)
    T, H = 900, 8
    s = np.round(rng.standard_normal((T, H)) * 2).astype(np.float32) / 2          # a handful of distinct values
    s[rng.random((T, H)) < 0.05] = np.nan
    s[rng.random((T, H)) < 0.02] = np.inf
    s[rng.random((T, H)) < 0.02] = -np.inf
    s[::7, 3] = -0.0
    s[:, 5] = np.nan                                                              # a head with no number at all
    s[:, 6] = 1.0                                                                 # a head of one value
    lens = _run(binding, oracle, [T], H, 64, 32, 0.3, per_layer, s)
    if not per_layer:
        assert lens[0, 5] == 32 and lens[0, 6] == T        # nothing but the window; all tied, all kept


def test_topk_config2_size(binding, oracle):
    rng = np.random.default_rng(4)
    T, H = 32768, 8
    s = rng.standard_normal((T, H)).astype(np.float32)
    lens = _run(binding, oracle, [T], H, 128, 128, 0.25, False, s)
    assert (lens == 128 + int(np.ceil(np.float32(0.25) * (T - 128)))).all()
    lens = _run(binding, oracle, [T], H, 128, 128, 0.25, True, s)
    assert lens.sum() == H * (128 + int(np.ceil(np.float32(0.25) * (T - 128))))
