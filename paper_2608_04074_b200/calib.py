"""Offline host calibration (float64): transforms, equal-volume grouping, Lloyd codebooks.

This is the paper's calibration stage (Algorithm 1 lines 1-6, Algorithm 2, Algorithm 3,
Theorem 1, Corollary 1, Theorem 2).  It runs once per model on the host and produces the
tables that ``novakv_load_calibration`` hands to the GPU library; it is not on the decode or
append hot path and nothing here runs per token.

Conventions: row vectors, maps act on the right (App. A).  Per KV head the result holds

* ``rk``        R_K      = M_q^{1/2} E   (analysis, d x d), grouping folded into the columns
* ``rk_inv_t``  R_K^{-T} = M_q^{-1/2} E  (used on the query, and as the synthesis matrix)
* ``k_mean``    calibration key mean
* ``rv``        R_V = eigenvectors of M_o (orthogonal), grouping folded into the columns
* ``v_mean``    calibration value mean (Remark after Corollary 1: centring values is exact)
* ``cb_k``, ``cb_v``  L = d/g codebooks of 256 centroids in R^g

Readings where the paper leaves a choice (stated again in the design notes):
rank r (0-based, decreasing variance) goes to group r mod L (Fig. "groupings" (c)); inside a
group coordinates keep rank order; for values the sort key is the measured variance of the
transform coefficients on the calibration values; eigenvector signs are fixed so that the
entry of largest magnitude is positive; k-means is seeded with distinct training vectors and
runs a fixed number of iterations; the per-token scale of Algorithm 3 is off (it is outside
Theorem 2's model and would break the exact 2 bits/element).
Value codebooks are finally snapped to a 7-bit grid per (KV head, group, coordinate) (the paper
stores its codebooks in a narrow format offline as well): encoder, decoder and oracle therefore see
the same centroids, and the decode kernel can keep a value codeword in four bytes.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass, field

import numpy as np

from . import build as _build

EIG_FLOOR = 1e-30  # App. A "Calibration statistics": eigenvalues of M_q floored, no ridge


@dataclass
class Calibration:
    """Per-layer calibration tables, float32 at the library boundary."""

    head_dim: int
    group_size: int
    codebook_size: int
    rk: np.ndarray         # [Hkv][d][d]
    rk_inv_t: np.ndarray   # [Hkv][d][d]
    rv: np.ndarray         # [Hkv][d][d]
    k_mean: np.ndarray     # [Hkv][d]
    v_mean: np.ndarray     # [Hkv][d]
    cb_k: np.ndarray       # [Hkv][L][C][g]
    cb_v: np.ndarray       # [Hkv][L][C][g]
    info: dict = field(default_factory=dict)

    @property
    def n_kv_heads(self) -> int:
        return self.rk.shape[0]

    @property
    def n_groups(self) -> int:
        return self.head_dim // self.group_size


def _sym_eig_desc(a: np.ndarray) -> tuple[np.ndarray, np.ndarray]:
    w, e = np.linalg.eigh((a + a.T) * 0.5)
    order = np.argsort(-w, kind="stable")
    w, e = w[order], e[:, order]
    # fix signs: largest-magnitude entry of each eigenvector positive
    idx = np.argmax(np.abs(e), axis=0)
    sgn = np.sign(e[idx, np.arange(e.shape[1])])
    sgn[sgn == 0] = 1.0
    return w, e * sgn


def msqrt_pair(mq: np.ndarray) -> tuple[np.ndarray, np.ndarray]:
    """Symmetric M_q^{1/2} and M_q^{-1/2} with eigenvalues floored at 1e-30 (App. A)."""
    w, u = np.linalg.eigh((mq + mq.T) * 0.5)
    w = np.maximum(w, EIG_FLOOR)
    return (u * np.sqrt(w)) @ u.T, (u / np.sqrt(w)) @ u.T


def key_transform(q_heads: np.ndarray, k: np.ndarray):
    """Algorithm 2 lines 1-4 for one KV head.

    q_heads: [N][H][d] queries of the H heads sharing this KV head; k: [M][d] keys.
    Returns (R_K, R_K^{-T}, k_mean, lambda) before any grouping.
    """
    d = k.shape[1]
    qq = q_heads.reshape(-1, d)
    mq = qq.T @ qq                                    # summed over the shared heads (App. F, GQA)
    k_mean = k.mean(axis=0)
    kc = k - k_mean
    sk = kc.T @ kc
    mh, mih = msqrt_pair(mq)
    lam, e = _sym_eig_desc(mh @ sk @ mh)
    return mh @ e, mih @ e, k_mean, lam


def attention_outputs(q: np.ndarray, k: np.ndarray, v: np.ndarray) -> np.ndarray:
    """Textbook softmax attention of every query over the whole (k, v) set (Eq. "scores")."""
    d = k.shape[1]
    z = (q @ k.T) / np.sqrt(d)
    z -= z.max(axis=1, keepdims=True)
    p = np.exp(z)
    p /= p.sum(axis=1, keepdims=True)
    return p @ v


def value_transform(o: np.ndarray):
    """Corollary 1: R_V = eigenvectors (decreasing eigenvalue) of M_o = sum_i o_i^T o_i."""
    mo = o.T @ o
    lam, e = _sym_eig_desc(mo)
    return e, lam


def equalizing_order(variances: np.ndarray, n_groups: int) -> np.ndarray:
    """Column order that folds the equal-volume grouping of Sec. 4 into a transform.

    Coordinates are ranked by decreasing variance (stable: the lower original index first on
    equal keys); rank r is dealt to group r mod L.  The returned permutation lists, for group
    0, 1, ..., L-1 in turn, the original coordinates of ranks l, l+L, l+2L, ...
    """
    d = variances.shape[0]
    g = d // n_groups
    rank_to_coord = np.argsort(-variances, kind="stable")
    order = np.empty(d, dtype=np.int64)
    for l in range(n_groups):
        for m in range(g):
            order[l * g + m] = rank_to_coord[l + m * n_groups]
    return order


GRID_LEVELS = 127          # a value-codebook coordinate takes the values lo + u (hi - lo) / 127, u = 0 .. 127


def snap_to_byte_grid(cb: np.ndarray) -> np.ndarray:
    """Round every codebook coordinate to its own 7-bit grid and return float32 values.

    cb: [..][C][g].  Coordinate i of a codebook takes the values lo_i + u (hi_i - lo_i) / 127, u = 0 .. 127,
    where lo_i / hi_i are the smallest / largest float32 value of that coordinate over the C codewords; the
    grid is evaluated in float64 and rounded once to float32 (``novakv_load_calibration`` re-derives the
    grid from the snapped values with the same arithmetic and refuses anything else).
    """
    cb32 = np.asarray(cb, dtype=np.float32)
    lo = cb32.min(axis=-2, keepdims=True).astype(np.float64)
    hi = cb32.max(axis=-2, keepdims=True).astype(np.float64)
    step = (hi - lo) / float(GRID_LEVELS)
    step = np.where(step > 0, step, 1.0)
    u = np.clip(np.rint((cb32.astype(np.float64) - lo) / step), 0, GRID_LEVELS)
    return (lo + step * u).astype(np.float32)


def _lloyd_c(x_groups: np.ndarray, init: np.ndarray, iters: int):
    lib = ctypes.CDLL(str(_build.build_calib_host()))
    fn = lib.novakv_calib_lloyd
    fn.restype = None
    fn.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_long, ctypes.c_int, ctypes.c_void_p,
                   ctypes.c_int, ctypes.c_int, ctypes.c_void_p]
    x = np.ascontiguousarray(x_groups, dtype=np.float64)
    c = np.ascontiguousarray(init, dtype=np.float64).copy()
    n_groups, n, g = x.shape
    k = c.shape[1]
    dist = np.zeros((n_groups, iters), dtype=np.float64)
    fn(x.ctypes.data, n_groups, n, g, c.ctypes.data, k, iters, dist.ctypes.data)
    return c, dist


def train_codebooks(coef: np.ndarray, n_groups: int, codebook_size: int, iters: int,
                    gen: np.random.Generator):
    """Algorithm 3 (per-token scale off): one codebook per group of g consecutive columns.

    coef: [M][d] transform coefficients with the grouping already folded into the columns.
    Returns (codebooks [L][C][g] float64, distortion trace [L][iters]).
    """
    m, d = coef.shape
    g = d // n_groups
    x = np.ascontiguousarray(coef.reshape(m, n_groups, g).transpose(1, 0, 2))
    init = np.empty((n_groups, codebook_size, g))
    for l in range(n_groups):
        # random-distinct initialisation: distinct training vectors, seeded
        uniq = np.unique(x[l], axis=0)
        if uniq.shape[0] < codebook_size:
            raise ValueError("fewer distinct training vectors than codewords")
        pick = gen.choice(uniq.shape[0], size=codebook_size, replace=False)
        init[l] = uniq[np.sort(pick)]
    return _lloyd_c(x, init, iters)


def calibrate(q_cal: np.ndarray, k_cal: np.ndarray, v_cal: np.ndarray, *, n_kv_heads: int,
              group_size: int = 4, codebook_size: int = 256, lloyd_iters: int = 25,
              seed: int = 0, n_q_for_values: int | None = None,
              snap_value_codebook: bool = True, key_scale: bool = False) -> Calibration:
    """Run the whole offline calibration for one layer.

    q_cal: [N][Hq][d], k_cal / v_cal: [M][Hkv][d] (float64).
    n_q_for_values bounds how many calibration queries per head form M_o (cost is N*M*d).
    key_scale: train the key codebooks on RMS-normalised coefficients r / rho, rho = ||r|| / sqrt(d)
    (Algorithm 3, "Normalize"), for the key format that stores a per-token scale.
    """
    n, hq, d = q_cal.shape
    hg = hq // n_kv_heads
    n_groups = d // group_size
    gen = np.random.Generator(np.random.PCG64(seed))
    out = dict(rk=[], rk_inv_t=[], rv=[], k_mean=[], v_mean=[], cb_k=[], cb_v=[])
    info = dict(key_lambda=[], key_coef_var=[], value_coef_var=[], key_distortion=[],
                value_distortion=[])
    for kvh in range(n_kv_heads):
        qh = q_cal[:, kvh * hg:(kvh + 1) * hg, :]
        k = k_cal[:, kvh, :]
        v = v_cal[:, kvh, :]
        # ---- keys (Theorem 1, Algorithm 2)
        rk, rk_inv_t, k_mean, lam = key_transform(qh, k)
        coef = (k - k_mean) @ rk
        var_k = coef.var(axis=0)                      # equals lambda / M up to rounding
        order = equalizing_order(var_k, n_groups)
        rk, rk_inv_t = rk[:, order], rk_inv_t[:, order]
        coef = coef[:, order]
        if key_scale:
            rho = np.sqrt((coef * coef).mean(axis=1, keepdims=True))
            coef = coef / np.where(rho > 0, rho, 1.0)
        cb_k, dist_k = train_codebooks(coef, n_groups, codebook_size, lloyd_iters, gen)
        # ---- values (Corollary 1)
        nq = n if n_q_for_values is None else min(n, n_q_for_values)
        o = np.concatenate([attention_outputs(qh[:nq, h, :], k, v) for h in range(hg)], axis=0)
        rv, _ = value_transform(o)
        v_mean = v.mean(axis=0)
        coef_v = (v - v_mean) @ rv
        var_v = coef_v.var(axis=0)
        order_v = equalizing_order(var_v, n_groups)
        rv = rv[:, order_v]
        coef_v = coef_v[:, order_v]
        cb_v, dist_v = train_codebooks(coef_v, n_groups, codebook_size, lloyd_iters, gen)
        out["rk"].append(rk); out["rk_inv_t"].append(rk_inv_t); out["rv"].append(rv)
        out["k_mean"].append(k_mean); out["v_mean"].append(v_mean)
        out["cb_k"].append(cb_k); out["cb_v"].append(cb_v)
        info["key_lambda"].append(lam); info["key_coef_var"].append(var_k[order])
        info["value_coef_var"].append(var_v[order_v])
        info["key_distortion"].append(dist_k); info["value_distortion"].append(dist_v)
    f32 = {name: np.ascontiguousarray(np.stack(vals), dtype=np.float32) for name, vals in out.items()}
    if snap_value_codebook:
        unsnapped = f32["cb_v"]
        f32["cb_v"] = snap_to_byte_grid(unsnapped)
        info["value_snap_rms"] = np.sqrt(((f32["cb_v"].astype(np.float64) - unsnapped) ** 2).mean(axis=(1, 2, 3)))
        info["value_codeword_rms"] = np.sqrt((unsnapped.astype(np.float64) ** 2).mean(axis=(1, 2, 3)))
    extra = {k_: info.pop(k_) for k_ in ("value_snap_rms", "value_codeword_rms") if k_ in info}
    info = {k_: np.stack(v_) for k_, v_ in info.items()}
    info.update(extra)
    info["lloyd_iters"] = lloyd_iters
    info["seed"] = seed
    return Calibration(head_dim=d, group_size=group_size, codebook_size=codebook_size, info=info,
                       **f32)
