"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU oracle harness.

This module holds *no arithmetic of the method*: it only draws random numbers with the
shapes and statistics of the paper's workloads (Sec. 5 and App. B describe keys, values
and queries of Qwen3-8B- and GPT-OSS-20B-shaped attention layers; App. D reports spectra
that decay over many decades; App. J reports heavy-tailed key channels).  Everything is a
pure function of an integer seed, so the CUDA path and the oracle can be fed bit-identical
inputs without sharing any code of their own.

Recipe (all draws come from ``numpy.random.Generator(PCG64(seed))``):

* a covariance per role (key, value, each query head):  ``U diag(i^-1.5) U^T`` with ``U`` the
  Q-factor of a seeded Gaussian matrix, i = 1..d;
* tokens are zero-mean Gaussian with that covariance;
* optional key outlier channels: ``n_outlier`` seeded channels whose samples are multiplied
  by 10 in the identity basis after sampling;
* optional heavy-tailed key channels: a seeded fraction of channels is replaced by
  Student-t (nu = 4) variates scaled to that channel's Gaussian standard deviation;
* queries are scaled by one scalar per KV head so that the standard deviation of
  ``q.k / sqrt(d)`` over the drawn samples is ``logit_std`` (otherwise attention is uniform
  and a relative tolerance on the output tests nothing);
* ragged lengths are ``clip(round(exp(N(ln median, sigma^2))), lo, hi)``;
* page tables are a seeded permutation of the physical page ids.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

__all__ = [
    "LayerShape",
    "rng",
    "decaying_covariance_factor",
    "draw_tokens",
    "draw_layer_laws",
    "LayerLaws",
    "draw_kv",
    "draw_q",
    "lognormal_lengths",
    "shuffled_page_table",
    "to_bf16_representable",
]


@dataclass(frozen=True)
class LayerShape:
    """Attention-layer geometry: query heads, KV heads, head dimension."""

    n_q_heads: int
    n_kv_heads: int
    head_dim: int

    @property
    def hg(self) -> int:
        return self.n_q_heads // self.n_kv_heads


def rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(int(seed)))


def decaying_covariance_factor(gen: np.random.Generator, d: int, power: float = 1.5) -> np.ndarray:
    """Return F (d x d) such that x = z F with z ~ N(0, I) has covariance U diag(i^-power) U^T."""
    a = gen.standard_normal((d, d))
    u, _ = np.linalg.qr(a)
    spec = np.arange(1, d + 1, dtype=np.float64) ** (-power)
    return (np.sqrt(spec)[:, None] * u.T)  # rows: sqrt(lambda_i) u_i^T


def draw_tokens(gen: np.random.Generator, factor: np.ndarray, n: int) -> np.ndarray:
    z = gen.standard_normal((n, factor.shape[0]))
    return z @ factor


@dataclass
class LayerLaws:
    """Per-head sampling laws of one synthetic layer."""

    shape: LayerShape
    key_factor: np.ndarray      # [Hkv][d][d]
    value_factor: np.ndarray    # [Hkv][d][d]
    query_factor: np.ndarray    # [Hq][d][d]
    outlier_channels: np.ndarray  # [Hkv][n_outlier] int
    heavy_channels: np.ndarray    # [Hkv][n_heavy] int
    query_gain: np.ndarray      # [Hkv] scalar applied to the queries of that KV head


def draw_layer_laws(
    shape: LayerShape,
    seed: int,
    n_outlier: int = 0,
    heavy_fraction: float = 0.0,
    logit_std: float = 3.0,
    power: float = 1.5,
) -> LayerLaws:
    gen = rng(seed)
    d = shape.head_dim
    kf = np.stack([decaying_covariance_factor(gen, d, power) for _ in range(shape.n_kv_heads)])
    vf = np.stack([decaying_covariance_factor(gen, d, power) for _ in range(shape.n_kv_heads)])
    qf = np.stack([decaying_covariance_factor(gen, d, power) for _ in range(shape.n_q_heads)])
    out_ch = np.stack(
        [gen.permutation(d)[:n_outlier] for _ in range(shape.n_kv_heads)]
    ).astype(np.int64).reshape(shape.n_kv_heads, n_outlier)
    n_heavy = int(round(heavy_fraction * d))
    heavy_ch = np.stack(
        [gen.permutation(d)[:n_heavy] for _ in range(shape.n_kv_heads)]
    ).astype(np.int64).reshape(shape.n_kv_heads, n_heavy)
    laws = LayerLaws(shape, kf, vf, qf, out_ch, heavy_ch, np.ones(shape.n_kv_heads))
    # Query gain: measured on a small seeded probe so that std(q.k/sqrt(d)) == logit_std.
    probe = rng(seed + 7919)
    gains = np.ones(shape.n_kv_heads)
    for kvh in range(shape.n_kv_heads):
        k = _draw_keys_one_head(probe, laws, kvh, 512)
        zs = []
        for h in range(kvh * shape.hg, (kvh + 1) * shape.hg):
            q = draw_tokens(probe, qf[h], 64)
            zs.append((q @ k.T).ravel() / np.sqrt(d))
        gains[kvh] = logit_std / np.std(np.concatenate(zs))
    laws.query_gain = gains
    return laws


def _draw_keys_one_head(gen: np.random.Generator, laws: LayerLaws, kvh: int, n: int) -> np.ndarray:
    k = draw_tokens(gen, laws.key_factor[kvh], n)
    hc = laws.heavy_channels[kvh]
    if hc.size:
        std = np.sqrt(np.sum(laws.key_factor[kvh][:, hc] ** 2, axis=0))
        t = gen.standard_t(4.0, size=(n, hc.size))
        k[:, hc] = t * std
    oc = laws.outlier_channels[kvh]
    if oc.size:
        k[:, oc] *= 10.0
    return k


def draw_kv(laws: LayerLaws, seed: int, n_tokens: int) -> tuple[np.ndarray, np.ndarray]:
    """Keys and values, float64, shape [n_tokens][Hkv][d]."""
    gen = rng(seed)
    s = laws.shape
    k = np.empty((n_tokens, s.n_kv_heads, s.head_dim))
    v = np.empty((n_tokens, s.n_kv_heads, s.head_dim))
    for kvh in range(s.n_kv_heads):
        k[:, kvh, :] = _draw_keys_one_head(gen, laws, kvh, n_tokens)
        v[:, kvh, :] = draw_tokens(gen, laws.value_factor[kvh], n_tokens)
    return k, v


def draw_q(laws: LayerLaws, seed: int, n: int) -> np.ndarray:
    """Queries, float64, shape [n][Hq][d]."""
    gen = rng(seed)
    s = laws.shape
    q = np.empty((n, s.n_q_heads, s.head_dim))
    for h in range(s.n_q_heads):
        q[:, h, :] = draw_tokens(gen, laws.query_factor[h], n) * laws.query_gain[h // s.hg]
    return q


def lognormal_lengths(seed: int, n: int, median: int = 8192, sigma: float = 1.0,
                      lo: int = 1024, hi: int = 131072) -> np.ndarray:
    gen = rng(seed)
    x = np.exp(gen.normal(np.log(median), sigma, size=n))
    return np.clip(np.rint(x), lo, hi).astype(np.int32)


def shuffled_page_table(seed: int, seq_lens: np.ndarray, page_tokens: int,
                        max_pages_per_seq: int | None = None) -> tuple[np.ndarray, int]:
    """Assign distinct physical pages to every sequence in a seeded random order.

    Returns (page_table int32 [n_seq][max_pages_per_seq] filled with -1 where unused,
    number of physical pages used).
    """
    gen = rng(seed)
    need = (np.asarray(seq_lens, dtype=np.int64) + page_tokens - 1) // page_tokens
    mp = int(need.max()) if max_pages_per_seq is None else int(max_pages_per_seq)
    total = int(need.sum())
    ids = gen.permutation(total).astype(np.int32)
    table = np.full((len(seq_lens), mp), -1, dtype=np.int32)
    pos = 0
    for b, n in enumerate(need):
        table[b, :n] = ids[pos:pos + n]
        pos += int(n)
    return table, total


def to_bf16_representable(x: np.ndarray) -> np.ndarray:
    """Round float values to the nearest bfloat16 (ties to even), returned as float32.

    Queries and newly appended keys/values are bf16 at the library boundary; both the CUDA
    path and the oracle receive these rounded values.
    """
    a = np.ascontiguousarray(x, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)
