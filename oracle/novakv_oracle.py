"""ctypes wrapper around the float64 CPU oracle (TEST INFRASTRUCTURE ONLY).

Only the tests, the smoke check and the benchmark's CPU-baseline / reference arm may import
this module.  It builds ``novakv_oracle.c`` with gcc next to the source and exposes the
oracle's functions on numpy arrays.  It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_DIR = Path(__file__).resolve().parent
_SRC = _DIR / "novakv_oracle.c"
_LIB = _DIR / "libnovakv_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    if not force and _LIB.exists() and _LIB.stat().st_mtime >= _SRC.stat().st_mtime:
        return _LIB
    flags = ["-O2", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC"]
    try:
        with open("/proc/cpuinfo") as f:
            if " fma " in f.read():
                flags.append("-mfma")     # fmaf() becomes one instruction; results are identical
    except OSError:
        pass
    res = subprocess.run(["gcc", *flags, str(_SRC), "-lm", "-o", str(_LIB)],
                         capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("gcc failed building the oracle:\n" + res.stdout + res.stderr)
    return _LIB


class _Tables(ctypes.Structure):
    _fields_ = [("n_kv_heads", ctypes.c_int), ("head_dim", ctypes.c_int),
                ("group_size", ctypes.c_int), ("codebook_size", ctypes.c_int),
                ("rk", ctypes.c_void_p), ("rk_inv_t", ctypes.c_void_p), ("rv", ctypes.c_void_p),
                ("k_mean", ctypes.c_void_p), ("v_mean", ctypes.c_void_p),
                ("cb_k", ctypes.c_void_p), ("cb_v", ctypes.c_void_p)]


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(str(build()))
        for name in ("oracle_coefficients", "oracle_search", "oracle_encode", "oracle_reconstruct",
                     "oracle_attention", "oracle_decode"):
            getattr(_lib, name).restype = None
    return _lib


def cpu_threads() -> int:
    """Threads the oracle's OpenMP loops will use (affinity-limited core count)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env)
    return len(os.sched_getaffinity(0))


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _u8(a):
    return np.ascontiguousarray(a, dtype=np.uint8)


class Oracle:
    """The oracle bound to one layer's calibration tables (float32 values widened to float64)."""

    def __init__(self, rk, rk_inv_t, rv, k_mean, v_mean, cb_k, cb_v):
        self.rk, self.rk_inv_t, self.rv = _f64(rk), _f64(rk_inv_t), _f64(rv)
        self.k_mean, self.v_mean = _f64(k_mean), _f64(v_mean)
        self.cb_k, self.cb_v = _f64(cb_k), _f64(cb_v)
        self.n_kv_heads, self.d = self.rk.shape[0], self.rk.shape[1]
        self.n_groups, self.codebook_size, self.g = self.cb_k.shape[1:]
        assert self.n_groups * self.g == self.d
        self._t = _Tables(self.n_kv_heads, self.d, self.g, self.codebook_size,
                          self.rk.ctypes.data, self.rk_inv_t.ctypes.data, self.rv.ctypes.data,
                          self.k_mean.ctypes.data, self.v_mean.ctypes.data,
                          self.cb_k.ctypes.data, self.cb_v.ctypes.data)

    @classmethod
    def from_calibration(cls, cal):
        return cls(cal.rk, cal.rk_inv_t, cal.rv, cal.k_mean, cal.v_mean, cal.cb_k, cal.cb_v)

    # -- write path -------------------------------------------------------------------
    def coefficients(self, x, which: str):
        """(x - mean) R for x of shape [n][Hkv][d]; which in {"k", "v"}."""
        x = _f64(x)
        n = x.shape[0]
        out = np.empty_like(x)
        m, mean = (self.rk, self.k_mean) if which == "k" else (self.rv, self.v_mean)
        lib = _load()
        for j in range(n):
            for h in range(self.n_kv_heads):
                lib.oracle_coefficients(ctypes.c_void_p(x[j, h].ctypes.data),
                                        ctypes.c_void_p(mean[h].ctypes.data),
                                        ctypes.c_void_p(m[h].ctypes.data), self.d,
                                        ctypes.c_void_p(out[j, h].ctypes.data))
        return out

    def search(self, coef, kvh: int, which: str):
        """Nearest-codeword search of given coefficients [n][d] against one head's codebooks.

        Returns (idx, float64 relative gap between the two nearest codewords), each [n][L].
        """
        coef = _f64(coef)
        n = coef.shape[0]
        cb = (self.cb_k if which == "k" else self.cb_v)[kvh]
        idx = np.empty((n, self.n_groups), np.uint8)
        gap = np.empty((n, self.n_groups), np.float64)
        _load().oracle_search(ctypes.c_void_p(coef.ctypes.data), ctypes.c_long(n), self.d, self.g,
                              self.codebook_size, ctypes.c_void_p(cb.ctypes.data),
                              ctypes.c_void_p(idx.ctypes.data), ctypes.c_void_p(gap.ctypes.data))
        return idx, gap

    def encode(self, k, v, with_gaps: bool = True):
        """k, v: [n][Hkv][d] -> dict(kidx, vidx[, kgap, vgap]), each [n][Hkv][L]."""
        k, v = _f64(k), _f64(v)
        n = k.shape[0]
        shp = (n, self.n_kv_heads, self.n_groups)
        res = dict(kidx=np.empty(shp, np.uint8), vidx=np.empty(shp, np.uint8))
        if with_gaps:
            res.update(kgap=np.empty(shp, np.float64), vgap=np.empty(shp, np.float64))

        def p(name):
            return ctypes.c_void_p(res[name].ctypes.data) if name in res else ctypes.c_void_p(0)

        _load().oracle_encode(ctypes.byref(self._t), ctypes.c_void_p(k.ctypes.data),
                              ctypes.c_void_p(v.ctypes.data), ctypes.c_long(n), p("kidx"), p("vidx"),
                              p("kgap"), p("vgap"))
        return res

    def key_scale(self, coef):
        """Per-token scale of coefficient vectors [n][d] (Algorithm "Codebook training", Normalize):
        returns (rho [n] float32 holding bfloat16 values, normalised coefficients [n][d])."""
        coef = _f64(coef)
        n, d = coef.shape
        rho = np.empty(n, np.float32)
        out = np.empty_like(coef)
        lib = _load()
        lib.oracle_key_scale.restype = ctypes.c_float
        for j in range(n):
            rho[j] = lib.oracle_key_scale(ctypes.c_void_p(coef[j].ctypes.data), d,
                                          ctypes.c_void_p(out[j].ctypes.data))
        return rho, out

    def encode_scaled(self, k, v, with_gaps: bool = True):
        """Write path of the scaled key format: as encode(), plus kscale [n][Hkv] (float32 holding
        bfloat16 values)."""
        k, v = _f64(k), _f64(v)
        n = k.shape[0]
        shp = (n, self.n_kv_heads, self.n_groups)
        res = dict(kidx=np.empty(shp, np.uint8), vidx=np.empty(shp, np.uint8),
                   kscale=np.empty((n, self.n_kv_heads), np.float32))
        if with_gaps:
            res.update(kgap=np.empty(shp, np.float64), vgap=np.empty(shp, np.float64))

        def p(name):
            return ctypes.c_void_p(res[name].ctypes.data) if name in res else ctypes.c_void_p(0)

        _load().oracle_encode_scaled(ctypes.byref(self._t), ctypes.c_void_p(k.ctypes.data),
                                     ctypes.c_void_p(v.ctypes.data), ctypes.c_long(n), p("kidx"), p("vidx"),
                                     p("kscale"), p("kgap"), p("vgap"))
        return res

    def reconstruct_scaled(self, kidx, vidx, kscale):
        """Explicit dequantisation of the scaled key format: k_hat = rho * Q(.) R_K^{-1} + k_mean."""
        kidx, vidx = _u8(kidx), _u8(vidx)
        kscale = np.ascontiguousarray(kscale, np.float32)
        s = kidx.shape[0]
        k_hat = np.empty((s, self.n_kv_heads, self.d))
        v_hat = np.empty((s, self.n_kv_heads, self.d))
        _load().oracle_reconstruct_scaled(ctypes.byref(self._t), ctypes.c_void_p(kidx.ctypes.data),
                                          ctypes.c_void_p(vidx.ctypes.data), ctypes.c_void_p(kscale.ctypes.data),
                                          ctypes.c_long(s), ctypes.c_void_p(k_hat.ctypes.data),
                                          ctypes.c_void_p(v_hat.ctypes.data))
        return k_hat, v_hat

    def decode_scaled(self, q, kidx, vidx, kscale, sm_scale: float | None = None):
        """One decode step of one sequence on the scaled key format."""
        q = _f64(q)
        kidx, vidx = _u8(kidx), _u8(vidx)
        kscale = np.ascontiguousarray(kscale, np.float32)
        hq = q.shape[0]
        s = kidx.shape[0]
        scale = 1.0 / np.sqrt(self.d) if sm_scale is None else float(sm_scale)
        out = np.empty((hq, self.d))
        _load().oracle_decode_scaled(ctypes.byref(self._t), ctypes.c_void_p(q.ctypes.data),
                                     ctypes.c_void_p(kidx.ctypes.data), ctypes.c_void_p(vidx.ctypes.data),
                                     ctypes.c_void_p(kscale.ctypes.data), ctypes.c_long(s), hq,
                                     ctypes.c_double(scale), ctypes.c_void_p(out.ctypes.data))
        return out

    # -- read path --------------------------------------------------------------------
    def reconstruct(self, kidx, vidx):
        """Explicit dequantisation: indices [S][Hkv][L] -> (k_hat, v_hat) [S][Hkv][d]."""
        kidx, vidx = _u8(kidx), _u8(vidx)
        s = kidx.shape[0]
        k_hat = np.empty((s, self.n_kv_heads, self.d))
        v_hat = np.empty((s, self.n_kv_heads, self.d))
        _load().oracle_reconstruct(ctypes.byref(self._t), ctypes.c_void_p(kidx.ctypes.data),
                                   ctypes.c_void_p(vidx.ctypes.data), ctypes.c_long(s),
                                   ctypes.c_void_p(k_hat.ctypes.data), ctypes.c_void_p(v_hat.ctypes.data))
        return k_hat, v_hat

    def decode(self, q, kidx, vidx, sm_scale: float | None = None):
        """One decode step of one sequence: q [Hq][d], indices [S][Hkv][L] -> out [Hq][d]."""
        q = _f64(q)
        kidx, vidx = _u8(kidx), _u8(vidx)
        hq = q.shape[0]
        s = kidx.shape[0]
        scale = 1.0 / np.sqrt(self.d) if sm_scale is None else float(sm_scale)
        out = np.empty((hq, self.d))
        _load().oracle_decode(ctypes.byref(self._t), ctypes.c_void_p(q.ctypes.data),
                              ctypes.c_void_p(kidx.ctypes.data), ctypes.c_void_p(vidx.ctypes.data),
                              ctypes.c_long(s), hq, ctypes.c_double(scale),
                              ctypes.c_void_p(out.ctypes.data))
        return out

    # -- scalar INT2 value codec of the deployed format ------------------------------------
    def encode_values_int2(self, v):
        """v [n][Hkv][d] -> (codes uint8 [n][Hkv][d] in 0..3, meta float32 [n][Hkv][2] = (scale, zero),
        both bfloat16 values)."""
        v = _f64(v)
        n = v.shape[0]
        codes = np.empty((n, self.n_kv_heads, self.d), np.uint8)
        meta = np.empty((n, self.n_kv_heads, 2), np.float32)
        _load().oracle_encode_values_int2(ctypes.byref(self._t), ctypes.c_void_p(v.ctypes.data), ctypes.c_long(n),
                                          ctypes.c_void_p(codes.ctypes.data), ctypes.c_void_p(meta.ctypes.data))
        return codes, meta

    def reconstruct_values_int2(self, codes, meta):
        codes = _u8(codes)
        meta = np.ascontiguousarray(meta, np.float32)
        s = codes.shape[0]
        v_hat = np.empty((s, self.n_kv_heads, self.d))
        _load().oracle_reconstruct_values_int2(ctypes.byref(self._t), ctypes.c_void_p(codes.ctypes.data),
                                               ctypes.c_void_p(meta.ctypes.data), ctypes.c_long(s),
                                               ctypes.c_void_p(v_hat.ctypes.data))
        return v_hat

    def decode_deployed(self, q, kidx, kscale, vcodes, vmeta, k_exact=None, v_exact=None, band_mask=None,
                        sink=None, sm_scale: float | None = None):
        """Decode step on the deployed format: scaled vector-quantised keys, INT2 scalar values, optionally a
        BF16 band (exact rows where band_mask is set) and a sink logit.  Explicit dequantisation, then
        textbook attention."""
        kidx = _u8(kidx)
        dummy_v = np.zeros_like(kidx)
        k_hat, _ = self.reconstruct_scaled(kidx, dummy_v, kscale)
        v_hat = self.reconstruct_values_int2(vcodes, vmeta)
        if band_mask is not None:
            band_mask = np.asarray(band_mask, bool)
            k_hat[band_mask] = _f64(k_exact)[band_mask]
            v_hat[band_mask] = _f64(v_exact)[band_mask]
        if k_hat.shape[0] == 0:
            return np.zeros((np.asarray(q).shape[0], self.d))
        if sink is None:
            return attention(q, k_hat, v_hat, sm_scale)
        return attention_sink(q, k_hat, v_hat, sink, sm_scale)

    def decode_sink(self, q, kidx, vidx, sink, kscale=None, sm_scale: float | None = None):
        """Decode step with a learned sink logit per query head (sink [Hq], natural-log units)."""
        q = _f64(q)
        kidx, vidx = _u8(kidx), _u8(vidx)
        sink = _f64(sink)
        ks = None if kscale is None else np.ascontiguousarray(kscale, np.float32)
        hq = q.shape[0]
        s = kidx.shape[0]
        scale = 1.0 / np.sqrt(self.d) if sm_scale is None else float(sm_scale)
        out = np.empty((hq, self.d))
        _load().oracle_decode_sink(ctypes.byref(self._t), ctypes.c_void_p(q.ctypes.data),
                                   ctypes.c_void_p(kidx.ctypes.data), ctypes.c_void_p(vidx.ctypes.data),
                                   ctypes.c_void_p(ks.ctypes.data if ks is not None else 0), ctypes.c_long(s), hq,
                                   ctypes.c_double(scale), ctypes.c_void_p(sink.ctypes.data),
                                   ctypes.c_void_p(out.ctypes.data))
        return out

    def decode_banded(self, q, kidx, vidx, k_exact, v_exact, band_mask, kscale=None, sink=None,
                      sm_scale: float | None = None):
        """Decode step on a cache whose tokens are partly held exactly (Fig. "Cache layout at decoding
        position t": the first n_sink and the most recent n_rec tokens stay in BF16, the tokens in between
        are quantised).  Every position is dequantised explicitly; positions with band_mask[j] set take the
        exact (bf16-representable) key and value instead; textbook attention follows.

        kidx, vidx [S][Hkv][L] (entries at band positions are ignored), k_exact / v_exact [S][Hkv][d],
        band_mask bool [S]."""
        band_mask = np.asarray(band_mask, bool)
        if kscale is None:
            k_hat, v_hat = self.reconstruct(kidx, vidx)
        else:
            k_hat, v_hat = self.reconstruct_scaled(kidx, vidx, kscale)
        k_hat[band_mask] = _f64(k_exact)[band_mask]
        v_hat[band_mask] = _f64(v_exact)[band_mask]
        if k_hat.shape[0] == 0:
            return np.zeros((np.asarray(q).shape[0], self.d))
        if sink is None:
            return attention(q, k_hat, v_hat, sm_scale)
        return attention_sink(q, k_hat, v_hat, sink, sm_scale)


def attention_sink(q, k, v, sink, sm_scale: float | None = None):
    """Textbook attention with an extra value-less logit per head: q [Hq][d], k/v [S][Hkv][d], sink [Hq]."""
    q, k, v, sink = _f64(q), _f64(k), _f64(v), _f64(sink)
    hq, d = q.shape
    s, hkv, _ = k.shape
    scale = 1.0 / np.sqrt(d) if sm_scale is None else float(sm_scale)
    out = np.empty((hq, d))
    _load().oracle_attention_sink(ctypes.c_void_p(q.ctypes.data), ctypes.c_void_p(k.ctypes.data),
                                  ctypes.c_void_p(v.ctypes.data), ctypes.c_long(s), hq, hkv, d,
                                  ctypes.c_double(scale), ctypes.c_void_p(sink.ctypes.data),
                                  ctypes.c_void_p(out.ctypes.data))
    return out


def attention(q, k, v, sm_scale: float | None = None):
    """Textbook attention on explicit float64 keys/values: q [Hq][d], k/v [S][Hkv][d]."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    hq, d = q.shape
    s, hkv, _ = k.shape
    scale = 1.0 / np.sqrt(d) if sm_scale is None else float(sm_scale)
    out = np.empty((hq, d))
    _load().oracle_attention(ctypes.c_void_p(q.ctypes.data), ctypes.c_void_p(k.ctypes.data),
                             ctypes.c_void_p(v.ctypes.data), ctypes.c_long(s), hq, hkv, d,
                             ctypes.c_double(scale), ctypes.c_void_p(out.ctypes.data))
    return out
