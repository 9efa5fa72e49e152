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
                 key_scale: bool = False, int2_values: bool = False):
        self.ctx = ctx
        self.key_scale = key_scale or int2_values
        self.int2_values = int2_values
        key_scale = self.key_scale
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
        # deployed format: scalar INT2 values with a bf16 (scale, zero) pair per token and KV head
        self.v_meta = (torch.zeros((self.n_pages, ctx.n_kv_heads, cache_format.PAGE_TOKENS, 2), dtype=torch.bfloat16,
                                   device=self.device) if int2_values else None)
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
    def load_value_meta(self, seq: int, pos0: int, n: int) -> np.ndarray:
        """(scale, zero) [n][Hkv][2] of positions pos0.. of one sequence."""
        mp = self.v_meta.float().cpu().numpy()
        pos = pos0 + np.arange(n)
        return mp[self.page_table_host[seq][pos // cache_format.PAGE_TOKENS], :, pos % cache_format.PAGE_TOKENS, :]

    def store_value_meta(self, seq: int, pos0: int, meta: np.ndarray):
        mp = self.v_meta.float().cpu().numpy()
        pos = pos0 + np.arange(meta.shape[0])
        mp[self.page_table_host[seq][pos // cache_format.PAGE_TOKENS], :, pos % cache_format.PAGE_TOKENS, :] = meta
        self.v_meta.copy_(torch.from_numpy(mp).to(torch.bfloat16))

    def append(self, layer, k_new, v_new, tok_seq, tok_pos):
        if self.int2_values:
            self.ctx.novakv_encode_append_deployed(layer, k_new, v_new, tok_seq, tok_pos, self.k_pages, self.v_pages,
                                                   self.k_scales, self.v_meta, self.page_table, self.seq_lens)
            return
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
        if self.int2_values:
            self.ctx.novakv_decode_attention_deployed(layer, q, self.k_pages, self.v_pages, self.k_scales, self.v_meta,
                                                      sink_logits, self.page_table, self.seq_lens, None, None, 0, None,
                                                      out, self.workspace, sm_scale)
            return out
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


class BandedCache:
    """Index cache plus a BF16 sink-plus-recent band: the first ``n_sink`` tokens of a sequence and its most
    recent ``n_rec`` .. ``n_rec + block - 1`` tokens stay in bf16; whenever the recent ring has grown by
    ``block`` tokens the ``block`` oldest are quantised into the index cache (deferred quantisation in
    blocks of eight steps).  Only bookkeeping and tensor copies happen here; encoding and attention are
    the library's calls."""

    def __init__(self, ctx: Context, batch: int, capacity_tokens: int, n_sink: int = 64, n_rec: int = 256,
                 block: int = 8, seed: int = 0, device="cuda:0", key_scale: bool = False, int2_values: bool = False):
        assert n_sink % cache_format.PAGE_TOKENS == 0
        self.ctx, self.batch, self.n_sink, self.n_rec, self.block = ctx, batch, n_sink, n_rec, block
        self.device = torch.device(device)
        self.paged = PagedCache(ctx, np.zeros(batch, np.int32), capacity_tokens=np.full(batch, capacity_tokens, np.int32),
                                seed=seed, device=device, key_scale=key_scale, int2_values=int2_values)
        self.ring_cap = n_rec + block
        self.cap = n_sink + self.ring_cap
        shape = (batch, self.cap, ctx.n_kv_heads, ctx.head_dim)
        self.band_k = torch.zeros(shape, dtype=torch.bfloat16, device=self.device)
        self.band_v = torch.zeros(shape, dtype=torch.bfloat16, device=self.device)
        self.total = np.zeros(batch, np.int64)          # tokens of each sequence
        self.quant = np.zeros(batch, np.int64)          # of which quantised (positions n_sink .. n_sink + quant - 1)
        self.ring_start = np.zeros(batch, np.int64)
        self.ring_len = np.zeros(batch, np.int64)
        self.band_meta = torch.zeros((batch, 3), dtype=torch.int32, device=self.device)
        self.quant_lens = torch.zeros(batch, dtype=torch.int32, device=self.device)
        self._staging = None

    def _sync_meta(self):
        meta = np.stack([np.minimum(self.total, self.n_sink), self.ring_start, self.ring_len], axis=1).astype(np.int32)
        self.band_meta.copy_(torch.from_numpy(meta))
        self.quant_lens.copy_(torch.from_numpy(self.quant.astype(np.int32)))

    def _flush(self, layer, items):
        """items: list of (b, n_tokens): quantise the n oldest ring tokens of sequence b."""
        ks, vs, seqs, poss = [], [], [], []
        for b, n in items:
            slots = self.n_sink + (self.ring_start[b] + np.arange(n)) % self.ring_cap
            idx = torch.from_numpy(slots).to(self.device)
            ks.append(self.band_k[b, idx]); vs.append(self.band_v[b, idx])
            seqs.append(np.full(n, b, np.int32))
            poss.append((self.n_sink + self.quant[b] + np.arange(n)).astype(np.int32))
            self.ring_start[b] = (self.ring_start[b] + n) % self.ring_cap
            self.ring_len[b] -= n
            self.quant[b] += n
        if not ks:
            return
        self.paged.append(layer, torch.cat(ks).contiguous(), torch.cat(vs).contiguous(),
                          torch.from_numpy(np.concatenate(seqs)).to(self.device),
                          torch.from_numpy(np.concatenate(poss)).to(self.device))

    def prefill(self, layer, b: int, k: torch.Tensor, v: torch.Tensor):
        """Tokens 0 .. n-1 of an empty sequence b (bf16 [n][Hkv][d]): sink, quantised middle, recent ring."""
        assert self.total[b] == 0
        n = int(k.shape[0])
        ns = min(n, self.n_sink)
        self.band_k[b, :ns] = k[:ns]; self.band_v[b, :ns] = v[:ns]
        rest = n - ns
        nrec = min(rest, self.n_rec)
        nq = rest - nrec
        if nq > 0:
            self.paged.append(layer, k[ns:ns + nq].contiguous(), v[ns:ns + nq].contiguous(),
                              torch.full((nq,), b, dtype=torch.int32, device=self.device),
                              torch.arange(ns, ns + nq, dtype=torch.int32, device=self.device))
        if nrec > 0:
            self.band_k[b, self.n_sink:self.n_sink + nrec] = k[ns + nq:]
            self.band_v[b, self.n_sink:self.n_sink + nrec] = v[ns + nq:]
        self.total[b], self.quant[b], self.ring_start[b], self.ring_len[b] = n, nq, 0, nrec
        self._sync_meta()

    def append_step(self, layer, k_new: torch.Tensor, v_new: torch.Tensor, mirror: bool = True):
        """One new token for every sequence (bf16 [batch][Hkv][d]): ``novakv_band_append`` places it, encodes the
        blocks that leave the band and advances the device-side state.  ``mirror`` keeps the host copies of that
        state in step by the same rule (bookkeeping for tests; ``refresh_host_state`` reads them back instead)."""
        if self._staging is None:
            n = self.ctx.novakv_band_append_staging_bytes(self.batch, self.block)
            self._staging = torch.empty(n, dtype=torch.uint8, device=self.device)
        p = self.paged
        self.ctx.novakv_band_append(layer, k_new, v_new, self.band_k, self.band_v, self.n_sink, self.n_rec, self.block,
                                    self.band_meta, self.quant_lens, p.k_pages, p.v_pages, p.k_scales,
                                    p.v_meta if p.int2_values else None, p.page_table, p.seq_lens, self._staging)
        if not mirror:
            return
        self.ring_len += self.total >= self.n_sink
        self.total += 1
        fl = self.ring_len >= self.n_rec + self.block
        self.ring_start[fl] = (self.ring_start[fl] + self.block) % self.ring_cap
        self.ring_len[fl] -= self.block
        self.quant[fl] += self.block

    def refresh_host_state(self):
        """Host copies of the band state from the device (after steps taken with ``mirror=False``)."""
        meta, quant = self.device_state()
        self.ring_start[:] = meta[:, 1]
        self.ring_len[:] = meta[:, 2]
        self.quant[:] = quant
        self.total[:] = meta[:, 0].astype(np.int64) + quant + meta[:, 2]

    def device_state(self):
        """(sink_cnt, ring_start, ring_len) [batch][3] and the quantised lengths [batch] as the device holds them."""
        return self.band_meta.cpu().numpy(), self.quant_lens.cpu().numpy()

    def band_mask(self, b: int) -> np.ndarray:
        """bool [total[b]]: positions held in bf16."""
        pos = np.arange(self.total[b])
        return (pos < self.n_sink) | (pos >= self.n_sink + self.quant[b])

    def decode(self, layer, q, out=None, sm_scale=None, sink_logits=None):
        if out is None:
            out = torch.empty((self.batch, self.ctx.n_q_heads, self.ctx.head_dim), dtype=torch.float32,
                              device=self.device)
        p = self.paged
        if p.int2_values:
            self.ctx.novakv_decode_attention_deployed(layer, q, p.k_pages, p.v_pages, p.k_scales, p.v_meta, sink_logits,
                                                      p.page_table, self.quant_lens, self.band_k, self.band_v,
                                                      self.n_sink, self.band_meta, out, p.workspace, sm_scale)
            return out
        self.ctx.novakv_decode_attention_banded(layer, q, p.k_pages, p.v_pages, p.k_scales, sink_logits, p.page_table,
                                                self.quant_lens, self.band_k, self.band_v, self.n_sink,
                                                self.band_meta, out, p.workspace, sm_scale)
        return out


def bf16_tensor(x: np.ndarray, device="cuda:0") -> torch.Tensor:
    """float array holding bf16-representable values -> torch bf16 tensor on the device."""
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16).to(device)
