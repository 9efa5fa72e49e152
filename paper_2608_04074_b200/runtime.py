"""Device-memory plumbing around the C-ABI library: paged pools, page tables, workspaces.

Nothing here computes any step of the method; tensors are allocated with torch and handed to
the kernels through ``binding.Context``.
"""
from __future__ import annotations

import numpy as np
import torch

from . import cache_format, synth
from .binding import Context


class PagedCache:
    """Key/value index pools plus page table and lengths for a batch of sequences."""

    def __init__(self, ctx: Context, seq_lens, capacity_tokens=None, seed: int = 0, device="cuda:0",
                 key_scale: bool = False):
        self.ctx = ctx
        self.key_scale = key_scale
        self.device = torch.device(device)
        seq_lens = np.asarray(seq_lens, dtype=np.int32)
        cap = seq_lens if capacity_tokens is None else np.maximum(np.asarray(capacity_tokens, np.int32), seq_lens)
        cap = np.maximum(cap, 1)
        table, n_pages = synth.shuffled_page_table(seed, cap, cache_format.PAGE_TOKENS)
        self.n_pages = max(int(n_pages), 1)
        self.page_table_host = table
        self.page_bytes = ctx.novakv_page_bytes()
        self.k_pages = torch.zeros((self.n_pages, self.page_bytes), dtype=torch.uint8, device=self.device)
        self.v_pages = torch.zeros((self.n_pages, self.page_bytes), dtype=torch.uint8, device=self.device)
        # scaled key format: one bf16 scale per token and KV head, [n_pages][Hkv][64]
        self.k_scales = (torch.ones((self.n_pages, ctx.n_kv_heads, cache_format.PAGE_TOKENS), dtype=torch.bfloat16,
                                    device=self.device) if key_scale else None)
        # unused table entries point at page 0 so that a wrong read stays in bounds
        self.page_table = torch.from_numpy(np.where(table < 0, 0, table).astype(np.int32)).to(self.device)
        self.seq_lens = torch.from_numpy(seq_lens.copy()).to(self.device)
        self.batch = int(len(seq_lens))
        self.workspace = torch.empty(ctx.novakv_decode_workspace_bytes(self.batch), dtype=torch.uint8,
                                     device=self.device)

    # ---- host-side packing of logical indices (tests fill a cache with the oracle's indices)
    def store_logical(self, seq: int, pos0: int, kidx: np.ndarray, vidx: np.ndarray):
        kp = self.k_pages.cpu().numpy().reshape(self.n_pages, self.ctx.n_kv_heads, -1)
        vp = self.v_pages.cpu().numpy().reshape(self.n_pages, self.ctx.n_kv_heads, -1)
        cache_format.write_tokens(kp, vp, self.page_table_host[seq], pos0, kidx, vidx)
        self.k_pages.copy_(torch.from_numpy(kp.reshape(self.n_pages, -1)))
        self.v_pages.copy_(torch.from_numpy(vp.reshape(self.n_pages, -1)))

    def store_logical_batch(self, items):
        """items: iterable of (seq, pos0, kidx, vidx); one round trip for all of them."""
        kp = self.k_pages.cpu().numpy().reshape(self.n_pages, self.ctx.n_kv_heads, -1)
        vp = self.v_pages.cpu().numpy().reshape(self.n_pages, self.ctx.n_kv_heads, -1)
        for seq, pos0, kidx, vidx in items:
            cache_format.write_tokens(kp, vp, self.page_table_host[seq], pos0, kidx, vidx)
        self.k_pages.copy_(torch.from_numpy(kp.reshape(self.n_pages, -1)))
        self.v_pages.copy_(torch.from_numpy(vp.reshape(self.n_pages, -1)))

    def load_logical(self, seq: int, pos0: int, n: int):
        kp = self.k_pages.cpu().numpy().reshape(self.n_pages, self.ctx.n_kv_heads, -1)
        vp = self.v_pages.cpu().numpy().reshape(self.n_pages, self.ctx.n_kv_heads, -1)
        return cache_format.read_tokens(kp, vp, self.page_table_host[seq], self.ctx.n_kv_heads,
                                        self.ctx.head_dim, pos0, n)

    def store_scales(self, seq: int, pos0: int, kscale: np.ndarray):
        """kscale [n][Hkv] (bf16-representable float32) -> scale pool, positions pos0.. of one sequence."""
        sp = self.k_scales.float().cpu().numpy()
        pos = pos0 + np.arange(kscale.shape[0])
        sp[self.page_table_host[seq][pos // cache_format.PAGE_TOKENS], :, pos % cache_format.PAGE_TOKENS] = kscale
        self.k_scales.copy_(torch.from_numpy(sp).to(torch.bfloat16))

    def load_scales(self, seq: int, pos0: int, n: int) -> np.ndarray:
        sp = self.k_scales.float().cpu().numpy()
        pos = pos0 + np.arange(n)
        return sp[self.page_table_host[seq][pos // cache_format.PAGE_TOKENS], :, pos % cache_format.PAGE_TOKENS]

    # ---- hot path calls
    def append(self, layer, k_new, v_new, tok_seq, tok_pos):
        if self.key_scale:
            self.ctx.novakv_encode_append_scaled(layer, k_new, v_new, tok_seq, tok_pos, self.k_pages, self.v_pages,
                                                 self.k_scales, self.page_table, self.seq_lens)
            return
        self.ctx.novakv_encode_append(layer, k_new, v_new, tok_seq, tok_pos, self.k_pages, self.v_pages,
                                      self.page_table, self.seq_lens)

    def decode(self, layer, q, out=None, sm_scale=None, sink_logits=None):
        if out is None:
            out = torch.empty((self.batch, self.ctx.n_q_heads, self.ctx.head_dim), dtype=torch.float32,
                              device=self.device)
        if sink_logits is not None:
            self.ctx.novakv_decode_attention_sink(layer, q, self.k_pages, self.v_pages, self.k_scales, sink_logits,
                                                  self.page_table, self.seq_lens, out, self.workspace, sm_scale)
            return out
        if self.key_scale:
            self.ctx.novakv_decode_attention_scaled(layer, q, self.k_pages, self.v_pages, self.k_scales,
                                                    self.page_table, self.seq_lens, out, self.workspace, sm_scale)
            return out
        self.ctx.novakv_decode_attention(layer, q, self.k_pages, self.v_pages, self.page_table, self.seq_lens,
                                         out, self.workspace, sm_scale)
        return out


def bf16_tensor(x: np.ndarray, device="cuda:0") -> torch.Tensor:
    """float array holding bf16-representable values -> torch bf16 tensor on the device."""
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16).to(device)
