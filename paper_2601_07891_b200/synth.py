"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds no arithmetic of the method: it only draws random tensors
(hidden states, surrogate weights, keys and values) and names the workload
shapes.  Both the CUDA path and the CPU oracle are fed from here, so that a
parity test compares the two on the very same bits.

Shapes follow the paper's three models (Appendix B, overhead table: H_Q, H, D,
D_h, D_int) and its surrogate sizes (Experiments, "KVzap training": input D_h,
hidden width D_h/8, output H = 8).  The paper's datasets and trained weights
are not used: inputs are i.i.d. normal draws, weights are N(0, 1/fan_in).
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np
import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    surrogate: str          # "linear" | "mlp"
    d_model: int
    hidden: int             # 0 for linear
    n_kv_heads: int
    head_dim: int
    n_layers: int
    batch: int
    seq_len: int            # tokens per sequence (prefill) / decode steps are separate
    tau: float
    window: int
    token_scale_sigma: float = 0.0   # log-normal per-token scale of the hidden states
    page_tokens: int = 0             # 0 = dense-ragged output
    decode_steps: int = 0
    prefix_min: int = 0
    prefix_max: int = 0


# The five configurations of the build's baseline file, in its order.
WORKLOADS = {
    "linear_4k": Workload("linear_4k", "linear", 4096, 0, 8, 128, 1, 1, 4096, 0.43, 128),
    "qwen3_8b_prefill_32k": Workload("qwen3_8b_prefill_32k", "mlp", 4096, 512, 8, 128, 36, 1, 32768, 0.43, 128),
    "llama31_8b_prefill_4x16k": Workload("llama31_8b_prefill_4x16k", "linear", 4096, 0, 8, 128, 32, 4, 16384,
                                         0.43, 128, token_scale_sigma=0.5),
    "qwen3_32b_prefill_128k_paged": Workload("qwen3_32b_prefill_128k_paged", "mlp", 5120, 640, 8, 128, 64, 1,
                                             131072, 0.43, 128, page_tokens=16),
    "qwen3_8b_decode_b128": Workload("qwen3_8b_decode_b128", "mlp", 4096, 512, 8, 128, 36, 128, 1, 0.43, 128,
                                     page_tokens=16, decode_steps=1024, prefix_min=4096, prefix_max=32768),
}
WORKLOAD_ORDER = ["linear_4k", "qwen3_8b_prefill_32k", "llama31_8b_prefill_4x16k",
                  "qwen3_32b_prefill_128k_paged", "qwen3_8b_decode_b128"]


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def hidden_states(n_tokens: int, d_model: int, seed: int, device="cpu",
                  token_scale_sigma: float = 0.0) -> torch.Tensor:
    """[n_tokens, d_model] bf16 ~ N(0,1), optionally times a per-token
    log-normal scale exp(sigma * N(0,1))."""
    g = _gen(seed, device)
    x = torch.randn(n_tokens, d_model, generator=g, device=device, dtype=torch.float32)
    if token_scale_sigma > 0.0:
        s = torch.randn(n_tokens, 1, generator=g, device=device, dtype=torch.float32)
        x = x * torch.exp(token_scale_sigma * s)
    return x.to(torch.bfloat16)


def _bias(n: int, sigma: float, g, device) -> torch.Tensor:
    if sigma > 0.0:
        return (sigma * torch.randn(n, generator=g, device=device, dtype=torch.float32)).contiguous()
    return torch.zeros(n, device=device, dtype=torch.float32)


def linear_weights(d_model: int, n_kv_heads: int, seed: int, device="cpu", bias_sigma: float = 0.0):
    """(W [H, d_model] bf16 ~ N(0, 1/d_model), b [H] fp32)."""
    g = _gen(seed, device)
    W = torch.randn(n_kv_heads, d_model, generator=g, device=device, dtype=torch.float32) / math.sqrt(d_model)
    return W.to(torch.bfloat16), _bias(n_kv_heads, bias_sigma, g, device)


def mlp_weights(d_model: int, hidden: int, n_kv_heads: int, seed: int, device="cpu", bias_sigma: float = 0.0):
    """(W1 [hidden, d_model] bf16, b1 [hidden] fp32, W2 [H, hidden] bf16, b2 [H] fp32),
    weights ~ N(0, 1/fan_in)."""
    g = _gen(seed, device)
    W1 = torch.randn(hidden, d_model, generator=g, device=device, dtype=torch.float32) / math.sqrt(d_model)
    W2 = torch.randn(n_kv_heads, hidden, generator=g, device=device, dtype=torch.float32) / math.sqrt(hidden)
    b1 = _bias(hidden, bias_sigma, g, device)
    b2 = _bias(n_kv_heads, bias_sigma, g, device)
    return W1.to(torch.bfloat16), b1, W2.to(torch.bfloat16), b2


def surrogate_weights(wl: Workload, layer: int, device="cpu", bias_sigma: float = 0.0, seed_base: int = 7000):
    seed = seed_base + layer
    if wl.surrogate == "linear":
        return linear_weights(wl.d_model, wl.n_kv_heads, seed, device, bias_sigma)
    return mlp_weights(wl.d_model, wl.hidden, wl.n_kv_heads, seed, device, bias_sigma)


def keys_values(n_kv_heads: int, n_tokens: int, head_dim: int, seed: int, device="cpu"):
    """(K, V), each [H, n_tokens, D] bf16 ~ N(0,1)."""
    g = _gen(seed, device)
    K = torch.randn(n_kv_heads, n_tokens, head_dim, generator=g, device=device, dtype=torch.float32)
    V = torch.randn(n_kv_heads, n_tokens, head_dim, generator=g, device=device, dtype=torch.float32)
    return K.to(torch.bfloat16), V.to(torch.bfloat16)


def cu_seqlens(lengths) -> np.ndarray:
    """Exclusive prefix of the per-sequence lengths, int32 [B+1]."""
    cu = np.zeros(len(lengths) + 1, dtype=np.int32)
    cu[1:] = np.cumsum(np.asarray(lengths, dtype=np.int64))
    return cu


def bits(t: torch.Tensor) -> np.ndarray:
    """Raw bf16 bit patterns of a tensor as a numpy uint16 array (on the host)."""
    assert t.dtype == torch.bfloat16
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def from_bits(a: np.ndarray, device="cpu") -> torch.Tensor:
    """Inverse of :func:`bits`."""
    assert a.dtype == np.uint16
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).to(device)


def quantize_e4m3(x: torch.Tensor, per_row: bool = True):
    """Input preparation for the 8-bit paths: x [rows, cols] (any float dtype) -> (bytes uint8 [rows, cols] of
    E4M3 values, scale fp32 [rows]) with x ~ scale[:, None] * E4M3(bytes); the scale maps each row's largest
    magnitude to 448, the format's largest value.  torch's own conversion does the rounding."""
    xf = x.to(torch.float32)
    amax = xf.abs().amax(dim=1) if per_row else xf.abs().max().expand(xf.shape[0])
    scale = torch.where(amax > 0, amax / 448.0, torch.ones_like(amax)).to(torch.float32).contiguous()
    q = (xf / scale[:, None]).to(torch.float8_e4m3fn)
    return q.view(torch.uint8).contiguous(), scale


E4M3_ROW_TRAILER = 16


def pack_rows_e4m3(x: torch.Tensor) -> torch.Tensor:
    """Input preparation for the 8-bit cache: x [..., D] (any float dtype) -> bf16 tensor [..., (D + 16) / 2] whose
    bytes are, per row, D E4M3 codes, the row's fp32 scale and 12 zero bytes (the row layout the 8-bit attention
    call reads; the other calls move such rows as opaque bytes)."""
    D = x.shape[-1]
    codes, scale = quantize_e4m3(x.reshape(-1, D))
    rows = torch.zeros(codes.shape[0], D + E4M3_ROW_TRAILER, dtype=torch.uint8, device=x.device)
    rows[:, :D] = codes
    rows[:, D:D + 4] = scale.view(torch.uint8).view(-1, 4)
    return rows.view(torch.bfloat16).view(*x.shape[:-1], (D + E4M3_ROW_TRAILER) // 2)


def unpack_rows_e4m3(bits: np.ndarray, D: int):
    """Rows as uint16 words [n, (D + 16) / 2] (a cache export, say) -> (codes uint8 [n, D], scale fp32 [n])."""
    raw = np.ascontiguousarray(bits).view(np.uint8).reshape(-1, D + E4M3_ROW_TRAILER)
    return np.ascontiguousarray(raw[:, :D]), np.ascontiguousarray(raw[:, D:D + 4]).view(np.float32).reshape(-1)
