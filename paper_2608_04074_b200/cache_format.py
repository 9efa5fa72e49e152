"""Fixed-width paged index cache: byte layout and rate accounting (host helpers, numpy only).

One uint8 codeword index per group of g = 4 transform coefficients, per token, per KV head,
for keys and for values (Sec. 2.2 "Quantization"; Sec. 5 "Bit rate"): L = d/4 bytes per
side, i.e. exactly 8/g = 2 bits per cached element.

Physical layout of a page (64 tokens), identical for every KV head:

* key pool    ``uint8 [n_pages][Hkv][64][L]``           token-major;
* value pool  ``uint8 [n_pages][Hkv][4][L][16]``        four 16-token blocks; inside a block one
  16-byte row per group (16 consecutive tokens), group ``g`` in row ``(g % 8) * (L // 8) + g // 8``
  (the decode kernel's tensor-core lanes then read their rows from distinct shared-memory banks).

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


def value_row_of_group(n_groups_: int) -> np.ndarray:
    """Row of each group inside a 16-token block of the value pool."""
    g = np.arange(n_groups_)
    return (g % 8) * (n_groups_ // 8) + g // 8


def index_bytes_per_token_per_kv_head(head_dim: int) -> int:
    """Key plus value index bytes of one token of one KV head."""
    return 2 * n_groups(head_dim)


def bits_per_element(head_dim: int, key_scale_bits: int = 0, value_meta_bits: int = 0) -> tuple[float, float]:
    """(key, value) cache rate in bits per stored element, optional per-token metadata bits."""
    l = n_groups(head_dim)
    return (8 * l + key_scale_bits) / head_dim, (8 * l + value_meta_bits) / head_dim


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
    """Store logical indices [n][Hkv][L] of one sequence at positions pos0.. into the pools."""
    n, hkv, l = kidx.shape
    kp = k_pool.reshape(k_pool.shape[0], hkv, PAGE_TOKENS, l)
    vp = v_pool.reshape(v_pool.shape[0], hkv, PAGE_TOKENS // V_BLOCK, l, V_BLOCK)
    pos = pos0 + np.arange(n)
    page = page_table_row[pos // PAGE_TOKENS]
    t = pos % PAGE_TOKENS
    for h in range(hkv):
        kp[page, h, t, :] = kidx[:, h, :]
        vp[page[:, None], h, (t // V_BLOCK)[:, None], value_row_of_group(l)[None, :], (t % V_BLOCK)[:, None]] = vidx[:, h, :]


def read_tokens(k_pool: np.ndarray, v_pool: np.ndarray, page_table_row: np.ndarray, n_kv_heads: int,
                head_dim: int, pos0: int, n: int) -> tuple[np.ndarray, np.ndarray]:
    """Logical indices [n][Hkv][L] of positions pos0 .. pos0+n-1 of one sequence."""
    l = n_groups(head_dim)
    kp = k_pool.reshape(k_pool.shape[0], n_kv_heads, PAGE_TOKENS, l)
    vp = v_pool.reshape(v_pool.shape[0], n_kv_heads, PAGE_TOKENS // V_BLOCK, l, V_BLOCK)
    pos = pos0 + np.arange(n)
    page = page_table_row[pos // PAGE_TOKENS]
    t = pos % PAGE_TOKENS
    kidx = np.empty((n, n_kv_heads, l), np.uint8)
    vidx = np.empty((n, n_kv_heads, l), np.uint8)
    for h in range(n_kv_heads):
        kidx[:, h, :] = kp[page, h, t, :]
        vidx[:, h, :] = vp[page[:, None], h, (t // V_BLOCK)[:, None], value_row_of_group(l)[None, :], (t % V_BLOCK)[:, None]]
    return kidx, vidx
