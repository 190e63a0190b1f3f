"""Shared helpers of the GPU parity tests: comparison rules, written once.

Rules (floating point decides an integer here, so the mask is compared in two
steps):
  * scores: |gpu - oracle| <= SCORE_ATOL (bf16 inputs, fp32 accumulation on
    the GPU, fp64 in the oracle);
  * keep mask implied by the GPU scores vs the oracle's: equal, except where
    the oracle score lies within SCORE_ATOL of tau;
  * lengths and compacted K/V: bit-exact against the oracle's mask + compaction
    run on the GPU's own fp32 scores (given the scores the result is unique);
  * rows past lengths keep the poison they were filled with.
"""
import numpy as np
import torch

from paper_2601_07891_b200 import synth

SCORE_ATOL = 2e-2
POISON = 0x7FC1          # a bf16 NaN pattern no input row contains


def dev(t):
    return t.cuda().contiguous() if t is not None else None


def weights_to_oracle(weights):
    out = []
    for i, w in enumerate(weights):
        if w is None:
            out.append(None)
        elif w.dtype == torch.bfloat16:
            out.append(synth.bits(w))
        else:
            out.append(w.detach().cpu().numpy())
    return tuple(out)


def check_scores(oracle, gpu_scores, X, weights, rows=None):
    """Compares GPU scores with the oracle on all rows or on a sample of rows."""
    Xb = synth.bits(X)
    got = gpu_scores.detach().cpu().numpy()
    if rows is not None:
        Xb = Xb[rows]
        got = got[rows]
    want = oracle.score(Xb, weights_to_oracle(weights))
    assert np.isfinite(got).all()
    err = np.abs(got - want).max() if got.size else 0.0
    assert err <= SCORE_ATOL, "score error %.3e exceeds %.1e" % (err, SCORE_ATOL)
    return want, float(err)


def check_mask_band(oracle, gpu_scores_np, oracle_scores_np, tau, w, cu):
    """Mask from GPU scores == mask from oracle scores outside the tolerance band."""
    keep_gpu = oracle.keep_mask(gpu_scores_np, tau, w, cu)
    keep_ref = oracle.keep_mask(oracle_scores_np, tau, w, cu)
    diff = keep_gpu != keep_ref                      # [H, T]
    if diff.any():
        near = np.abs(oracle_scores_np.T - np.float32(tau)) <= SCORE_ATOL
        assert not (diff & ~near).any(), "mask differs outside the tolerance band"
    return keep_gpu


def check_compaction(oracle, K, V, gpu_scores_np, tau, w, cu, K_out, V_out, lengths):
    """Bit-exact check of lengths and compacted rows given the GPU's scores."""
    Kb, Vb = synth.bits(K), synth.bits(V)
    keep = oracle.keep_mask(gpu_scores_np, tau, w, cu)
    K_ref, V_ref, len_ref = oracle.compact(Kb, Vb, keep, cu, fill=POISON)
    np.testing.assert_array_equal(lengths.cpu().numpy(), len_ref)
    np.testing.assert_array_equal(synth.bits(K_out), K_ref)      # includes the untouched (poison) rows
    np.testing.assert_array_equal(synth.bits(V_out), V_ref)
    return keep, len_ref


def poison_like(t):
    return torch.full_like(t.view(torch.int16), np.int16(POISON)).view(torch.bfloat16)
