"""Fixed-width paged index cache: byte layout and rate accounting (host helpers, numpy only).

One uint8 codeword index per group of g = 4 transform coefficients, per token, per KV head,
for keys and for values (Sec. 2.2 "Quantization"; Sec. 5 "Bit rate"): L = d/4 bytes per
side, i.e. exactly 8/g = 2 bits per cached element.

Physical layout: a page holds 64 tokens; per (page, KV head) one contiguous chunk of 64*L bytes
in the key pool and one in the value pool (``uint8 [n_pages][Hkv][64*L]`` each).  Inside a chunk
the bytes are ordered so that each lane of a decode warp loads, with one or two coalesced 128-bit
loads, exactly the bytes it consumes:

* keys:   ``[tile = t // 32][plane][t % 32][16 bytes]``.  Byte j of a token's L bytes holds the code
  of group ``j ^ (t % 8)`` for j < 16 and of group ``j ^ (t % 16)`` for j >= 16 (neighbouring lanes
  then read different columns of the score table at every step); plane = j // 16.
* values: ``[block = t // 16][fr = l % 8][fc = t % 4][gb = l // 8][b = (t % 16) // 4]``: the 16 (or
  8) bytes of MMA lane (fr, fc) are contiguous.

(t = token slot in the page, l = group.)

``page_table[seq][i]`` names the physical page that holds tokens ``64 i .. 64 i + 63``.
The functions below only permute bytes; they hold no arithmetic of the method.
"""
from __future__ import annotations

import numpy as np

PAGE_TOKENS = 64
V_BLOCK = 16
GROUP_SIZE = 4
CODEBOOK_SIZE = 256


def n_groups(head_dim: int) -> int:
    return head_dim // GROUP_SIZE


def key_offset(t, l, n_groups_: int):
    """Byte offset of (token slot t, group l) inside a key chunk (numpy arrays broadcast)."""
    kpl = n_groups_ // 16
    j = l ^ (t & np.where(np.asarray(l) < 16, 7, 15))
    return (((t >> 5) * kpl + (j >> 4)) * 32 + (t & 31)) * 16 + (j & 15)


def value_offset(t, l, n_groups_: int):
    """Byte offset of (token slot t, group l) inside a value chunk (numpy arrays broadcast)."""
    ngb = n_groups_ // 8
    tb = t & 15
    fc, b, fr = tb & 3, tb >> 2, l & 7
    return (t >> 4) * (n_groups_ * 16) + (fr * 4 + fc) * (ngb * 4) + ((l >> 3) ^ (fc & 1)) * 4 + b


def pack_int2(codes: np.ndarray) -> np.ndarray:
    """Scalar 2-bit codes [..][d] (0..3) -> one byte per group of 4: c0 | c1 << 2 | c2 << 4 | c3 << 6 ([..][d/4])."""
    c = np.asarray(codes, np.uint8).reshape(codes.shape[:-1] + (codes.shape[-1] // 4, 4))
    return (c[..., 0] | (c[..., 1] << 2) | (c[..., 2] << 4) | (c[..., 3] << 6)).astype(np.uint8)


def index_bytes_per_token_per_kv_head(head_dim: int) -> int:
    """Key plus value index bytes of one token of one KV head."""
    return 2 * n_groups(head_dim)


def bits_per_element(head_dim: int, key_scale_bits: int = 0, value_meta_bits: int = 0) -> tuple[float, float]:
    """(key, value) cache rate in bits per stored element, optional per-token metadata bits."""
    l = n_groups(head_dim)
    return (8 * l + key_scale_bits) / head_dim, (8 * l + value_meta_bits) / head_dim


def deployed_bits_per_element(context_tokens: int, head_dim: int = 128, n_sink: int = 64, n_rec: int = 256) -> float:
    """Average cache rate of the deployed format over keys and values at a given context length
    (Sec. 5 "Bit rate"): scaled 2-bit keys and INT2 values with their per-token metadata, and the
    n_sink + n_rec band tokens at 16 bits per element."""
    kb, vb = bits_per_element(head_dim, key_scale_bits=16, value_meta_bits=32)
    quant = 0.5 * (kb + vb)
    band = min(context_tokens, n_sink + n_rec)
    return quant + band * (16.0 - quant) / context_tokens


def table_scalars(head_dim: int, with_value_codebooks: bool = False) -> int:
    """Scalars stored once per (layer, KV head): 3 d^2 + d + L * 256 * g (+ value codebooks)."""
    l = n_groups(head_dim)
    n = 3 * head_dim * head_dim + head_dim + l * CODEBOOK_SIZE * GROUP_SIZE
    if with_value_codebooks:
        n += l * CODEBOOK_SIZE * GROUP_SIZE
    return n


def page_bytes(n_kv_heads: int, head_dim: int) -> int:
    """Bytes of one page of the key pool (= of the value pool), all KV heads."""
    return n_kv_heads * PAGE_TOKENS * n_groups(head_dim)


def alloc_pools(n_pages: int, n_kv_heads: int, head_dim: int) -> tuple[np.ndarray, np.ndarray]:
    shape = (n_pages, n_kv_heads, PAGE_TOKENS * n_groups(head_dim))
    return np.zeros(shape, np.uint8), np.zeros(shape, np.uint8)


def write_tokens(k_pool: np.ndarray, v_pool: np.ndarray, page_table_row: np.ndarray, pos0: int,
                 kidx: np.ndarray, vidx: np.ndarray) -> None:
    """Store logical indices [n][Hkv][L] of one sequence at positions pos0.. into the pools
    (pools shaped [n_pages][Hkv][64*L])."""
    n, hkv, l = kidx.shape
    pos = pos0 + np.arange(n)
    page = page_table_row[pos // PAGE_TOKENS][:, None]
    t = (pos % PAGE_TOKENS)[:, None]
    g = np.arange(l)[None, :]
    ko, vo = key_offset(t, g, l), value_offset(t, g, l)
    for h in range(hkv):
        k_pool[page, h, ko] = kidx[:, h, :]
        v_pool[page, h, vo] = vidx[:, h, :]


def read_tokens(k_pool: np.ndarray, v_pool: np.ndarray, page_table_row: np.ndarray, n_kv_heads: int,
                head_dim: int, pos0: int, n: int) -> tuple[np.ndarray, np.ndarray]:
    """Logical indices [n][Hkv][L] of positions pos0 .. pos0+n-1 of one sequence."""
    l = n_groups(head_dim)
    pos = pos0 + np.arange(n)
    page = page_table_row[pos // PAGE_TOKENS][:, None]
    t = (pos % PAGE_TOKENS)[:, None]
    g = np.arange(l)[None, :]
    ko, vo = key_offset(t, g, l), value_offset(t, g, l)
    kidx = np.empty((n, n_kv_heads, l), np.uint8)
    vidx = np.empty((n, n_kv_heads, l), np.uint8)
    for h in range(n_kv_heads):
        kidx[:, h, :] = k_pool[page, h, ko]
        vidx[:, h, :] = v_pool[page, h, vo]
    return kidx, vidx
