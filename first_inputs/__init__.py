"""Seeded synthetic inputs for the routed decoder: model shapes, random weights,
token ids, prompt lengths, skip masks and stand-in KV caches.

This module only draws numbers and arranges them; it evaluates no router, no layer
and no attention.  Both the CUDA library's harness and the host oracle's tests feed
from it so that the two sides see identical bytes.  Everything is numpy on the host
and deterministic in (seed, stream name, chunk index): a tensor is cut into fixed
chunks, each chunk has its own Philox counter-based stream, so threads can fill
chunks in any order.
"""
from __future__ import annotations

import hashlib
import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import asdict, dataclass

import numpy as np

_CHUNK = 1 << 22  # elements per independently seeded chunk


@dataclass(frozen=True)
class ModelShape:
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn_dim: int
    vocab: int
    rope_base: float = 10000.0
    rms_eps: float = 1e-5

    def asdict(self):
        return asdict(self)

    @property
    def q_dim(self):
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self):
        return self.n_kv_heads * self.head_dim

    def layer_params(self):
        return (self.q_dim + 2 * self.kv_dim) * self.d_model + self.d_model * self.q_dim + 3 * self.ffn_dim * self.d_model


# Llama-style shapes used by the workloads (architecture numbers are public model cards).
TINY = ModelShape(4, 256, 4, 4, 64, 688, 1024, 10000.0)
TINY_GQA = ModelShape(3, 256, 8, 2, 32, 352, 512, 10000.0)
LLAMA_1B = ModelShape(16, 2048, 32, 8, 64, 8192, 128256, 500000.0)
LLAMA_3B = ModelShape(28, 3072, 24, 8, 128, 8192, 128256, 500000.0)
LLAMA_8B = ModelShape(32, 4096, 32, 8, 128, 14336, 128256, 500000.0)


def _key(seed: int, stream: str, chunk: int) -> int:
    h = hashlib.blake2b(f"{seed}/{stream}/{chunk}".encode(), digest_size=16).digest()
    return int.from_bytes(h, "little")


def _rng(seed: int, stream: str, chunk: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=_key(seed, stream, chunk) % (1 << 128)))


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal(shape, std: float, seed: int, stream: str, bf16: bool = False, mean: float = 0.0,
           threads: int | None = None) -> np.ndarray:
    """N(mean, std^2) tensor; float32, or bfloat16 bits (uint16) when ``bf16``."""
    shape = tuple(int(s) for s in np.atleast_1d(shape))
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16 if bf16 else np.float32)
    nchunks = (n + _CHUNK - 1) // _CHUNK

    def fill(c):
        lo, hi = c * _CHUNK, min(n, (c + 1) * _CHUNK)
        x = _rng(seed, stream, c).standard_normal(hi - lo, dtype=np.float32)
        x *= np.float32(std)
        if mean:
            x += np.float32(mean)
        out[lo:hi] = f32_to_bf16_bits(x) if bf16 else x

    threads = threads or min(32, os.cpu_count() or 1)
    if nchunks <= 1 or threads <= 1:
        for c in range(nchunks):
            fill(c)
    else:
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(fill, range(nchunks)))
    return out.reshape(shape)


def make_weights(shape: ModelShape, seed: int, bf16: bool, std: float = 0.02, layers=None) -> dict:
    """Random-init decoder weights, PyTorch Linear layout [out][in].

    Matrices ~ N(0, std^2); norm gains ~ 1 + N(0, std^2) so a dropped gain shows.
    With ``bf16`` every value (gains included) is rounded to bfloat16 once: matrices
    come back as uint16 bit patterns, gains as the rounded values in float32.
    ``layers`` restricts which layers are materialised (others are None)."""
    s = shape
    L = s.n_layers
    layers = range(L) if layers is None else layers

    def mat(name, o, i):
        return normal((o, i), std, seed, name, bf16)

    def gain(name):
        g = normal((s.d_model,), std, seed, name, False, mean=1.0)
        return bf16_bits_to_f32(f32_to_bf16_bits(g)) if bf16 else g

    w = {"embed": mat("embed", s.vocab, s.d_model), "lm_head": mat("lm_head", s.vocab, s.d_model),
         "final_norm": gain("final_norm")}
    per = {k: [None] * L for k in ("attn_norm", "ffn_norm", "wq", "wk", "wv", "wo", "wg", "wu", "wd")}
    for l in layers:
        per["attn_norm"][l] = gain(f"attn_norm{l}")
        per["ffn_norm"][l] = gain(f"ffn_norm{l}")
        per["wq"][l] = mat(f"wq{l}", s.q_dim, s.d_model)
        per["wk"][l] = mat(f"wk{l}", s.kv_dim, s.d_model)
        per["wv"][l] = mat(f"wv{l}", s.kv_dim, s.d_model)
        per["wo"][l] = mat(f"wo{l}", s.d_model, s.q_dim)
        per["wg"][l] = mat(f"wg{l}", s.ffn_dim, s.d_model)
        per["wu"][l] = mat(f"wu{l}", s.ffn_dim, s.d_model)
        per["wd"][l] = mat(f"wd{l}", s.d_model, s.ffn_dim)
    w.update(per)
    return w


def tokens(shape_or_vocab, n: int, seed: int, stream: str = "tokens") -> np.ndarray:
    vocab = shape_or_vocab.vocab if isinstance(shape_or_vocab, ModelShape) else int(shape_or_vocab)
    return _rng(seed, stream).integers(0, vocab, size=n, dtype=np.int32)


def prompt_lengths(B: int, lo: int, hi: int, seed: int) -> np.ndarray:
    """Prompt lengths uniform over the integers lo..hi inclusive."""
    return _rng(seed, "prompt_lengths").integers(lo, hi + 1, size=B, dtype=np.int32)


# ---- skip masks: uint8 [B][L], 1 = keep.  Structure follows what the paper reports:
# first and last layers never skipped, skipping concentrated mid-stack, many layers
# all-or-nothing across a task (Sec. "Layer-wise Skipping Patterns", appendix table of
# per-layer skipping percentages).

def mask_skip_fraction(B: int, L: int, f_lo: float, f_hi: float, seed: int) -> np.ndarray:
    """Each sequence skips round(f*L) distinct layers drawn from 1..L-2, f ~ U[f_lo, f_hi]."""
    g = _rng(seed, "mask_fraction")
    m = np.ones((B, L), dtype=np.uint8)
    for b in range(B):
        k = int(round(float(g.uniform(f_lo, f_hi)) * L))
        k = min(k, max(L - 2, 0))
        if k:
            m[b, g.choice(np.arange(1, L - 1), size=k, replace=False)] = 0
    return m


def mask_bernoulli(B: int, L: int, keep_p: float, seed: int) -> np.ndarray:
    """Independent keep with probability keep_p; layers 0 and L-1 always kept."""
    g = _rng(seed, "mask_bernoulli")
    m = (g.random((B, L)) < keep_p).astype(np.uint8)
    m[:, 0] = 1
    m[:, L - 1] = 1
    return m


def mask_aligned(B: int, L: int, frac: float) -> np.ndarray:
    """All sequences skip the same round(frac*L) layers, a contiguous mid-stack block
    centred on the middle of the stack (first and last layer kept)."""
    k = min(int(round(frac * L)), max(L - 2, 0))
    m = np.ones((B, L), dtype=np.uint8)
    if k:
        start = max(1, min(L - 1 - k, (L - k) // 2))
        m[:, start:start + k] = 0
    return m


def mask_independent(B: int, L: int, frac: float, seed: int) -> np.ndarray:
    """Every sequence skips exactly round(frac*L) layers of its own choice from 1..L-2."""
    return mask_skip_fraction(B, L, frac, frac, seed)


def mask_unified(B: int, L: int, every: int) -> np.ndarray:
    """Input-agnostic preset: every sequence skips the same evenly spaced layers, every
    `every`-th one counted from layer 1 (first and last layer kept). The fixed-interval
    skipping strategy the paper compares against (Section 4, baselines)."""
    m = np.ones((B, L), dtype=np.uint8)
    if every > 0:
        for l in range(1, L - 1):
            if l % every == every - 1:
                m[:, l] = 0
    return m


def mask_random_shared(B: int, L: int, frac: float, seed: int) -> np.ndarray:
    """Input-agnostic preset: one random set of round(frac*L) layers from 1..L-2, the same
    for every sequence. The random skipping strategy the paper compares against."""
    g = _rng(seed, "mask_random_shared")
    k = min(int(round(frac * L)), max(L - 2, 0))
    m = np.ones((B, L), dtype=np.uint8)
    if k:
        m[:, g.choice(np.arange(1, L - 1), size=k, replace=False)] = 0
    return m


def synthetic_kv_rows(n_tokens: int, kv_dim: int, seed: int, stream: str, bf16: bool = True) -> np.ndarray:
    """Stand-in cache contents N(0,1) for one (layer, sequence, K-or-V): [n_tokens][kv_dim]."""
    return normal((n_tokens, kv_dim), 1.0, seed, stream, bf16)
