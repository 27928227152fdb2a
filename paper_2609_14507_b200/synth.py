"""Seeded synthetic inputs shared by the tests, the benchmark and the oracle-side checks.

This module holds none of the method's arithmetic: it only draws numbers and converts
float32 to bf16 bit patterns.  The paper's workloads are ShareGPT-prompted runs of three models
(Sec. 7.1); those prompts and weights are not used here.  Seeded N(0,1) tensors with the models'
attention shapes stand in for them.

bf16 tensors are NumPy ``uint16`` arrays of raw bit patterns on the host and ``torch.bfloat16``
tensors on the device.
"""
from dataclasses import dataclass

import numpy as np


def f32_to_bf16_bits(x):
    """float32 -> bf16 bit patterns, round-to-nearest-even (NaN not expected in inputs)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits):
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(rng, shape):
    """N(0,1) float32 draws rounded to bf16 bits."""
    return f32_to_bf16_bits(rng.standard_normal(size=shape, dtype=np.float32))


@dataclass(frozen=True)
class Shape:
    """Attention shape of one model family."""
    name: str
    kind: str            # "gqa" or "mla"
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    dim_qk: int
    dim_v: int
    scale: float

    @property
    def bytes_per_token(self):
        if self.kind == "mla":
            return 2 * self.dim_qk
        return 2 * self.n_kv_heads * (self.dim_qk + self.dim_v)


# Shapes of the models the paper evaluates (Sec. 7.1): Mixtral-8x7B and Qwen3-30B-A3B are GQA with
# head_dim 128; DeepSeek-V2-Lite caches a 512-wide latent plus a 64-wide rope part shared by its 16 heads.
MIXTRAL = Shape("mixtral-8x7b", "gqa", 32, 32, 8, 128, 128, 128 ** -0.5)
QWEN3 = Shape("qwen3-30b-a3b", "gqa", 48, 32, 4, 128, 128, 128 ** -0.5)
DSV2_LITE = Shape("deepseek-v2-lite", "mla", 27, 16, 1, 576, 512, 192 ** -0.5)
SMALL_GQA = Shape("small-gqa", "gqa", 1, 32, 4, 128, 128, 128 ** -0.5)


def host_kv(shape, n_tokens, seed):
    """(K [n][Hkv][dqk], V [n][Hkv][dv] or None for MLA) as bf16 bits, from one seed."""
    rng = np.random.default_rng(seed)
    k = normal_bf16(rng, (n_tokens, shape.n_kv_heads, shape.dim_qk))
    v = None if shape.kind == "mla" else normal_bf16(rng, (n_tokens, shape.n_kv_heads, shape.dim_v))
    return k, v


def host_q(shape, n_seqs, seed):
    """Q [n_seqs][Hq][dqk] bf16 bits."""
    rng = np.random.default_rng(seed)
    return normal_bf16(rng, (n_seqs, shape.n_q_heads, shape.dim_qk))


def ragged_lengths(seed, n_seqs, lo, hi):
    """Context lengths uniform in [lo, hi] (inclusive), as the 1M-token sweep draws them."""
    return np.random.default_rng(seed).integers(lo, hi + 1, size=n_seqs).astype(np.int64)


def device_kv(shape, n_tokens, seed, device="cuda:0"):
    """Device-side N(0,1) bf16 (K, V or None); the same bits reach the oracle by a D2H copy."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    k = torch.randn((n_tokens, shape.n_kv_heads, shape.dim_qk), generator=g, device=device,
                    dtype=torch.float32).to(torch.bfloat16)
    v = None
    if shape.kind != "mla":
        v = torch.randn((n_tokens, shape.n_kv_heads, shape.dim_v), generator=g, device=device,
                        dtype=torch.float32).to(torch.bfloat16)
    return k, v


def device_q(shape, n_seqs, seed, device="cuda:0"):
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return torch.randn((n_seqs, shape.n_q_heads, shape.dim_qk), generator=g, device=device,
                       dtype=torch.float32).to(torch.bfloat16)


def torch_bits(t):
    """torch.bfloat16 tensor (any device) -> NumPy uint16 bit patterns on the host."""
    import torch
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def bits_to_torch(bits, device="cpu"):
    """NumPy uint16 bf16 bits -> torch.bfloat16 tensor."""
    import torch
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(device)
