"""Shared set-up for the GPU parity tests: build a context from a workload, compare with the oracle."""
from __future__ import annotations

import numpy as np

from oracle import novakv_oracle as O
from paper_2608_04074_b200 import synth

REL_TOL = 2e-3          # max|delta| <= 2e-3 * ||o||_inf on float32 output (the stated decode tolerance)
NEAR_TIE = 1e-6         # index mismatches are allowed only where the oracle's float64 relative gap is below this


class Case:
    """Calibration + context + oracle for one layer shape."""

    def __init__(self, wl, n_layers=1, key_scale=False):
        from paper_2608_04074_b200.binding import Context
        self.wl = wl
        self.key_scale = key_scale
        self.laws = wl.laws()
        self.cal = wl.calibration(self.laws, key_scale=key_scale)
        self.oracle = O.Oracle.from_calibration(self.cal)
        s = wl.shape
        self.ctx = Context(s.n_q_heads, s.n_kv_heads, s.head_dim, n_layers=n_layers)
        for layer in range(n_layers):
            self.ctx.novakv_load_calibration(layer, self.cal)

    def draw(self, seed, n_tokens, n_queries):
        k, v = synth.draw_kv(self.laws, seed, n_tokens)
        q = synth.draw_q(self.laws, seed + 1, n_queries)
        return (synth.to_bf16_representable(k), synth.to_bf16_representable(v), synth.to_bf16_representable(q))


def check_indices(gpu_idx, enc, which):
    """GPU indices must equal the oracle's decision; any difference must be a float64 near-tie."""
    ref = enc[which + "idx"]
    gap = enc[which + "gap"]
    diff = gpu_idx != ref
    n_diff = int(diff.sum())
    n_near = int((gap <= NEAR_TIE).sum())
    bad = diff & (gap > NEAR_TIE)
    assert not bad.any(), (
        f"{which}: {int(bad.sum())} index mismatches outside the near-tie band "
        f"(min gap among them {gap[bad].min():.3e}); total mismatches {n_diff}")
    return n_diff, n_near


def check_output(out_gpu, out_ref):
    out_gpu = np.asarray(out_gpu, dtype=np.float64)
    scale = np.abs(out_ref).max()
    err = np.abs(out_gpu - out_ref).max()
    assert np.isfinite(out_gpu).all()
    assert err <= REL_TOL * scale, f"max|delta| {err:.3e} > {REL_TOL} * ||o||inf {scale:.3e} (ratio {err / scale:.3e})"
    return err / scale
