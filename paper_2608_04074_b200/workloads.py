"""The synthetic workloads the tests and the benchmark run (shapes from the paper's models).

Each workload names a layer shape, a batch of sequence lengths and the calibration budget.
They stand in for KV caches of Qwen3-8B (32 query / 8 KV heads, d = 128) and GPT-OSS-20B
(64 / 8, d = 64) captured on the paper's evaluation prompts, which are not available here;
only shapes and qualitative statistics are taken (see ``synth``).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from . import synth
from .calib import Calibration, calibrate

PAGE_TOKENS = 64


@dataclass
class Workload:
    name: str
    shape: synth.LayerShape
    seq_lens: np.ndarray                 # int32 [B]
    seed: int
    n_outlier: int = 0
    heavy_fraction: float = 0.0
    calib_tokens: int = 4096
    calib_queries_for_values: int = 1024
    lloyd_iters: int = 25
    logit_std: float = 3.0
    notes: str = ""
    extra: dict = field(default_factory=dict)

    @property
    def batch(self) -> int:
        return int(len(self.seq_lens))

    @property
    def n_groups(self) -> int:
        return self.shape.head_dim // 4

    def decode_index_bytes(self) -> int:
        """Packed K+V index bytes one decode step must read (2 bits per element)."""
        return int(np.sum(self.seq_lens.astype(np.int64)) * self.shape.n_kv_heads * 2 * self.n_groups)

    def laws(self) -> synth.LayerLaws:
        return synth.draw_layer_laws(self.shape, 1000 * self.seed + 1, n_outlier=self.n_outlier,
                                     heavy_fraction=self.heavy_fraction, logit_std=self.logit_std)

    def calibration(self, laws: synth.LayerLaws | None = None, key_scale: bool = False) -> Calibration:
        """key_scale: key codebooks trained on RMS-normalised coefficients (per-token scale format)."""
        laws = laws or self.laws()
        k, v = synth.draw_kv(laws, 1000 * self.seed + 2, self.calib_tokens)
        q = synth.draw_q(laws, 1000 * self.seed + 3, self.calib_tokens)
        return calibrate(q, k, v, n_kv_heads=self.shape.n_kv_heads, lloyd_iters=self.lloyd_iters,
                         seed=1000 * self.seed + 4, n_q_for_values=self.calib_queries_for_values,
                         key_scale=key_scale)


def tiny(seq_len: int = 1024, seed: int = 1) -> Workload:
    """Tiny oracle check: batch 1, one KV head with 4 query heads, d = 64, S = 1024."""
    return Workload("tiny_d64_S%d" % seq_len, synth.LayerShape(4, 1, 64),
                    np.array([seq_len], np.int32), seed, calib_tokens=4096,
                    calib_queries_for_values=4096, lloyd_iters=10)


def qwen3_8b(batch: int = 8, seq_len: int = 16384, seed: int = 2, calib_tokens: int = 8192,
             lloyd_iters: int = 12) -> Workload:
    """Qwen3-8B-shaped layer, a few key outlier channels (std x10)."""
    return Workload("qwen3_8b_B%d_S%d" % (batch, seq_len), synth.LayerShape(32, 8, 128),
                    np.full(batch, seq_len, np.int32), seed, n_outlier=4,
                    calib_tokens=calib_tokens, lloyd_iters=lloyd_iters)


def gpt_oss_20b(batch: int = 16, seq_len: int = 65536, seed: int = 4, calib_tokens: int = 8192,
                lloyd_iters: int = 12) -> Workload:
    """GPT-OSS-20B-shaped full-attention layer, 5 % heavy-tailed (Student-t, nu=4) key channels."""
    return Workload("gpt_oss_20b_B%d_S%d" % (batch, seq_len), synth.LayerShape(64, 8, 64),
                    np.full(batch, seq_len, np.int32), seed, heavy_fraction=0.05,
                    calib_tokens=calib_tokens, lloyd_iters=lloyd_iters)


def paged_mix(n_seq: int = 128, seed: int = 5, calib_tokens: int = 8192, lloyd_iters: int = 12,
              lo: int = 1024, hi: int = 131072, median: int = 8192) -> Workload:
    """Serving mix: ragged lognormal lengths, Qwen3-8B KV shape, 64-token pages."""
    lens = synth.lognormal_lengths(1000 * seed + 9, n_seq, median=median, sigma=1.0, lo=lo, hi=hi)
    return Workload("paged_mix_%dseq" % n_seq, synth.LayerShape(32, 8, 128), lens, seed,
                    n_outlier=4, calib_tokens=calib_tokens, lloyd_iters=lloyd_iters)
