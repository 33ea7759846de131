"""Seeded random tensors for the FreeCache hot path.

Value recipes:
  * Q, K, V (fresh rows and cache rows): N(0, 1) drawn in fp32, rounded to bf16.  Every row of
    the cache buffer is random, including rows beyond ``cache_len`` (the contract says such
    rows may hold anything).
  * logits: z[b, i, :] = sigma[b, i] * N(0, 1) in fp32 with sigma[b, i] ~ U(lo, hi), so that
    the per-position confidence is skewed across the block.
  * mask: a seeded choice of ``n_masked`` positions per batch element.
  * tok_ar: equals tok_dlm with probability ``p_agree`` per position, otherwise
    (tok_dlm + 1 + r) mod vocab with r >= 0 drawn from the seed (never equal to tok_dlm).

Small tensors are drawn with the CPU generator; multi-GB caches may be drawn on the GPU
(``device="cuda"``), in which case the slices that the oracle checks are copied back, so
both sides still see the same bits.  Nothing here computes any step of the method.
"""
from __future__ import annotations

import numpy as np
import torch


def seed_for(cfg_index: int, step: int = 0) -> int:
    return 21467 + 1000 * int(cfg_index) + int(step)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def make_kv_rows(shape, seed: int, device="cpu") -> torch.Tensor:
    """N(0,1) in fp32 rounded to bf16, any shape."""
    x = torch.randn(*shape, generator=_gen(seed, device), device=device, dtype=torch.float32)
    return x.to(torch.bfloat16)


def make_attn_inputs(n_layers, batch, n_q_heads, n_kv_heads, q_cap, head_dim, seed, device="cpu"):
    """(q [nl,B,Hq,q_cap,D], k_new [nl,B,Hkv,q_cap,D], v_new likewise), bf16."""
    q = make_kv_rows((n_layers, batch, n_q_heads, q_cap, head_dim), seed * 7 + 1, device)
    k = make_kv_rows((n_layers, batch, n_kv_heads, q_cap, head_dim), seed * 7 + 2, device)
    v = make_kv_rows((n_layers, batch, n_kv_heads, q_cap, head_dim), seed * 7 + 3, device)
    return q, k, v


def make_cache(n_layers, batch, n_kv_heads, capacity, head_dim, seed, device="cpu"):
    """(cache_k, cache_v) bf16 [NL,B,Hkv,Lcap,D]; drawn layer by layer to bound fp32 scratch."""
    shape = (n_layers, batch, n_kv_heads, capacity, head_dim)
    ck = torch.empty(shape, dtype=torch.bfloat16, device=device)
    cv = torch.empty(shape, dtype=torch.bfloat16, device=device)
    gk, gv = _gen(seed * 7 + 4, device), _gen(seed * 7 + 5, device)
    for layer in range(n_layers):
        ck[layer] = torch.randn(shape[1:], generator=gk, device=device, dtype=torch.float32)
        cv[layer] = torch.randn(shape[1:], generator=gv, device=device, dtype=torch.float32)
    return ck, cv


def make_logits(batch, block_len, vocab, sigma_range, seed, device="cpu") -> torch.Tensor:
    lo, hi = sigma_range
    g = _gen(seed * 7 + 6, device)
    sigma = lo + (hi - lo) * torch.rand(batch, block_len, 1, generator=g, device=device)
    z = torch.randn(batch, block_len, vocab, generator=g, device=device, dtype=torch.float32)
    return (z * sigma).contiguous()


def make_mask(batch, block_len, n_masked, seed) -> torch.Tensor:
    """uint8 [B, Lblk] with exactly n_masked ones per batch element (CPU tensor)."""
    rng = np.random.default_rng(seed * 7 + 0)
    m = np.zeros((batch, block_len), np.uint8)
    for b in range(batch):
        m[b, rng.choice(block_len, size=n_masked, replace=False)] = 1
    return torch.from_numpy(m)


def make_tok_ar(tok_dlm: torch.Tensor, p_agree: float, vocab: int, seed: int) -> torch.Tensor:
    """AR argmax stand-in: agrees with tok_dlm with probability p_agree per position."""
    t = tok_dlm.detach().cpu().numpy().astype(np.int64)
    rng = np.random.default_rng(seed * 7 + 9)
    agree = rng.random(t.shape) < p_agree
    r = rng.integers(0, max(vocab - 1, 1), size=t.shape)
    other = (t + 1 + r) % vocab
    other = np.where(other == t, (t + 1) % vocab, other)
    out = np.where(agree | (t < 0), t, other).astype(np.int32)
    return torch.from_numpy(out)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 bit patterns (CPU copy)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def widen(t: torch.Tensor) -> np.ndarray:
    """bf16 / fp32 tensor -> contiguous fp32 numpy array (exact widening)."""
    return t.detach().cpu().to(torch.float32).contiguous().numpy()
