"""Thin ctypes binding of libnovakv.so: argument marshalling only.

Every function mirrors the entry point of the same name in ``include/novakv.h`` and passes
``torch`` tensors as raw device pointers plus the current CUDA stream.  There is no CPU or
PyTorch fallback: if the shared library is missing or a call returns an error status, a
``NovaKVError`` is raised.
"""
from __future__ import annotations

import ctypes
from ctypes import c_int, c_float, c_void_p, c_size_t, c_long, c_double, c_uint32, POINTER

import numpy as np

from . import build as _build

EXPORTED = [
    "novakv_create", "novakv_destroy", "novakv_status_string", "novakv_load_calibration",
    "novakv_page_bytes", "novakv_decode_workspace_bytes", "novakv_encode_append",
    "novakv_decode_attention", "novakv_last_device_status", "novakv_step_staging_bytes",
    "novakv_step_host", "novakv_step_host_async", "novakv_search_coefficients", "novakv_bf16_workspace_bytes",
    "novakv_bf16_decode_attention", "novakv_profile_enable", "novakv_profile_read",
    "novakv_launch_count", "novakv_debug_set_scan_ctas", "novakv_decode_attention_noalloc", "novakv_debug_set_value_path",
    "novakv_scale_page_bytes", "novakv_encode_append_scaled", "novakv_decode_attention_scaled",
    "novakv_decode_attention_sink", "novakv_decode_attention_banded",
    "novakv_value_meta_page_bytes", "novakv_encode_append_deployed", "novakv_decode_attention_deployed",
    "novakv_debug_set_segment_weight", "novakv_debug_set_fused_merge",
    "novakv_band_append_staging_bytes", "novakv_band_append",
]


class NovaKVError(RuntimeError):
    pass


class Config(ctypes.Structure):
    _fields_ = [("n_layers", c_int), ("n_q_heads", c_int), ("n_kv_heads", c_int), ("head_dim", c_int),
                ("group_size", c_int), ("codebook_size", c_int), ("page_tokens", c_int), ("device", c_int)]


class CalibrationPtrs(ctypes.Structure):
    _fields_ = [(n, c_void_p) for n in ("rk", "rk_inv_t", "rv", "k_mean", "v_mean", "cb_k", "cb_v")]


_lib = None


NOALLOC_SCRATCH_BYTES = 4 << 20      # NOVAKV_NOALLOC_SCRATCH_BYTES of the public header


def load_library(path=None):
    """Load libnovakv.so (built in-tree by ``build.build_cuda``); raises if it is absent."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    import os
    p = str(path or os.environ.get("NOVAKV_LIB") or _build.LIB_CUDA)
    try:
        lib = ctypes.CDLL(p)
    except OSError as e:
        raise NovaKVError(f"cannot load {p}: build it with paper_2608_04074_b200.build.build_cuda() ({e})")
    lib.novakv_create.argtypes = [POINTER(c_void_p), POINTER(Config)]
    lib.novakv_destroy.argtypes = [c_void_p]
    lib.novakv_status_string.argtypes = [c_int]
    lib.novakv_status_string.restype = ctypes.c_char_p
    lib.novakv_load_calibration.argtypes = [c_void_p, c_int, POINTER(CalibrationPtrs)]
    lib.novakv_page_bytes.argtypes = [c_void_p]
    lib.novakv_page_bytes.restype = c_size_t
    lib.novakv_decode_workspace_bytes.argtypes = [c_void_p, c_int]
    lib.novakv_decode_workspace_bytes.restype = c_size_t
    lib.novakv_encode_append.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_int,
                                         c_void_p, c_void_p, c_int, c_void_p, c_int, c_int, c_void_p, c_void_p]
    lib.novakv_decode_attention.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_int, c_void_p,
                                            c_int, c_void_p, c_int, c_float, c_void_p, c_int, c_void_p,
                                            c_size_t, c_void_p]
    lib.novakv_scale_page_bytes.argtypes = [c_void_p]
    lib.novakv_scale_page_bytes.restype = c_size_t
    lib.novakv_encode_append_scaled.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_int,
                                                c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_int, c_int,
                                                c_void_p, c_void_p]
    lib.novakv_decode_attention_scaled.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_int,
                                                   c_void_p, c_int, c_void_p, c_int, c_float, c_void_p, c_int,
                                                   c_void_p, c_size_t, c_void_p]
    lib.novakv_decode_attention_sink.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                                 c_int, c_void_p, c_int, c_void_p, c_int, c_float, c_void_p, c_int,
                                                 c_void_p, c_size_t, c_void_p]
    lib.novakv_decode_attention_banded.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                                   c_int, c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_int, c_int,
                                                   c_void_p, c_int, c_float, c_void_p, c_int, c_void_p, c_size_t,
                                                   c_void_p]
    lib.novakv_value_meta_page_bytes.argtypes = [c_void_p]
    lib.novakv_value_meta_page_bytes.restype = c_size_t
    lib.novakv_encode_append_deployed.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_int,
                                                  c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_int,
                                                  c_int, c_void_p, c_void_p]
    lib.novakv_decode_attention_deployed.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                                     c_void_p, c_int, c_void_p, c_int, c_void_p, c_void_p, c_void_p,
                                                     c_int, c_int, c_void_p, c_int, c_float, c_void_p, c_int, c_void_p,
                                                     c_size_t, c_void_p]
    lib.novakv_band_append_staging_bytes.argtypes = [c_void_p, c_int, c_int]
    lib.novakv_band_append_staging_bytes.restype = c_size_t
    lib.novakv_band_append.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_int, c_int, c_int,
                                       c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p,
                                       c_int, c_void_p, c_void_p, c_size_t, c_void_p]
    lib.novakv_decode_attention_noalloc.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_int, c_void_p,
                                                    c_int, c_void_p, c_int, c_float, c_void_p, c_int, c_void_p]
    lib.novakv_last_device_status.argtypes = [c_void_p, c_void_p, POINTER(c_uint32)]
    lib.novakv_step_staging_bytes.argtypes = [c_void_p, c_int, c_int]
    lib.novakv_step_staging_bytes.restype = c_size_t
    lib.novakv_step_host_async.argtypes = lib.novakv_step_host.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p,
                                     c_void_p, c_void_p, c_int, c_void_p, c_int, c_void_p, c_int, c_float,
                                     c_void_p, c_void_p, c_size_t, c_void_p, c_size_t, c_void_p]
    lib.novakv_search_coefficients.argtypes = [c_void_p, c_int, c_int, c_void_p, c_int, c_void_p, c_void_p]
    lib.novakv_bf16_workspace_bytes.argtypes = [c_void_p, c_int, c_int]
    lib.novakv_bf16_workspace_bytes.restype = c_size_t
    lib.novakv_bf16_decode_attention.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_int,
                                                 c_void_p, c_int, c_float, c_int, c_void_p, c_int, c_void_p,
                                                 c_size_t, c_void_p]
    lib.novakv_profile_enable.argtypes = [c_void_p, c_int]
    lib.novakv_profile_read.argtypes = [c_void_p, c_int, POINTER(c_double), POINTER(c_long)]
    lib.novakv_launch_count.argtypes = [c_void_p]
    lib.novakv_debug_set_scan_ctas.argtypes = [c_void_p, c_int]
    lib.novakv_debug_set_value_path.argtypes = [c_void_p, c_int]
    lib.novakv_debug_set_segment_weight.argtypes = [c_void_p, c_int]
    lib.novakv_debug_set_fused_merge.argtypes = [c_void_p, c_int]
    lib.novakv_launch_count.restype = c_long
    if path is None:
        _lib = lib
    return lib


def _check(lib, status, what):
    if status != 0:
        raise NovaKVError(f"{what}: {lib.novakv_status_string(status).decode()} (status {status})")


def _ptr(t):
    return c_void_p(0) if t is None else c_void_p(t.data_ptr())


def _stream():
    import torch
    return c_void_p(torch.cuda.current_stream().cuda_stream)


class Context:
    """Owns a ``novakv_ctx``; methods carry the names of the C entry points."""

    def __init__(self, n_q_heads, n_kv_heads, head_dim, n_layers=1, device=0):
        self.lib = load_library()
        self.cfg = Config(n_layers, n_q_heads, n_kv_heads, head_dim, 4, 256, 64, device)
        self.handle = c_void_p()
        _check(self.lib, self.lib.novakv_create(ctypes.byref(self.handle), ctypes.byref(self.cfg)), "novakv_create")
        self.n_q_heads, self.n_kv_heads, self.head_dim = n_q_heads, n_kv_heads, head_dim
        self.n_groups = head_dim // 4

    def close(self):
        if self.handle:
            self.lib.novakv_destroy(self.handle)
            self.handle = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- tables -----------------------------------------------------------------------------
    def novakv_load_calibration(self, layer, cal):
        """cal: object with float32 numpy arrays rk, rk_inv_t, rv, k_mean, v_mean, cb_k, cb_v."""
        keep = {}
        ptrs = CalibrationPtrs()
        for name in ("rk", "rk_inv_t", "rv", "k_mean", "v_mean", "cb_k", "cb_v"):
            a = getattr(cal, name, None)
            if a is None:
                setattr(ptrs, name, None)
                continue
            a = np.ascontiguousarray(a, dtype=np.float32)
            keep[name] = a
            setattr(ptrs, name, a.ctypes.data)
        _check(self.lib, self.lib.novakv_load_calibration(self.handle, layer, ctypes.byref(ptrs)),
               "novakv_load_calibration")

    def novakv_page_bytes(self):
        return int(self.lib.novakv_page_bytes(self.handle))

    def novakv_decode_workspace_bytes(self, batch):
        return int(self.lib.novakv_decode_workspace_bytes(self.handle, batch))

    # -- hot path ---------------------------------------------------------------------------
    def novakv_encode_append(self, layer, k_new, v_new, tok_seq, tok_pos, k_pages, v_pages, page_table, seq_lens):
        n_tokens = int(k_new.shape[0]) if k_new is not None else 0
        _check(self.lib, self.lib.novakv_encode_append(
            self.handle, layer, _ptr(k_new), _ptr(v_new), _ptr(tok_seq), _ptr(tok_pos), n_tokens,
            _ptr(k_pages), _ptr(v_pages), int(k_pages.shape[0]), _ptr(page_table), int(page_table.shape[1]),
            int(page_table.shape[0]), _ptr(seq_lens), _stream()), "novakv_encode_append")

    def novakv_decode_attention(self, layer, q, k_pages, v_pages, page_table, seq_lens, out, workspace,
                                sm_scale=None):
        import torch
        batch = int(q.shape[0])
        scale = float(self.head_dim) ** -0.5 if sm_scale is None else float(sm_scale)
        _check(self.lib, self.lib.novakv_decode_attention(
            self.handle, layer, _ptr(q), _ptr(k_pages), _ptr(v_pages), int(k_pages.shape[0]), _ptr(page_table),
            int(page_table.shape[1]), _ptr(seq_lens), batch, scale, _ptr(out),
            1 if out.dtype == torch.float32 else 0, _ptr(workspace),
            int(workspace.numel() * workspace.element_size()), _stream()), "novakv_decode_attention")

    def novakv_scale_page_bytes(self):
        return int(self.lib.novakv_scale_page_bytes(self.handle))

    def novakv_encode_append_scaled(self, layer, k_new, v_new, tok_seq, tok_pos, k_pages, v_pages, k_scales,
                                    page_table, seq_lens):
        n_tokens = int(k_new.shape[0]) if k_new is not None else 0
        _check(self.lib, self.lib.novakv_encode_append_scaled(
            self.handle, layer, _ptr(k_new), _ptr(v_new), _ptr(tok_seq), _ptr(tok_pos), n_tokens,
            _ptr(k_pages), _ptr(v_pages), _ptr(k_scales), int(k_pages.shape[0]), _ptr(page_table),
            int(page_table.shape[1]), int(page_table.shape[0]), _ptr(seq_lens), _stream()),
            "novakv_encode_append_scaled")

    def novakv_decode_attention_scaled(self, layer, q, k_pages, v_pages, k_scales, page_table, seq_lens, out,
                                       workspace, sm_scale=None):
        import torch
        batch = int(q.shape[0])
        scale = float(self.head_dim) ** -0.5 if sm_scale is None else float(sm_scale)
        _check(self.lib, self.lib.novakv_decode_attention_scaled(
            self.handle, layer, _ptr(q), _ptr(k_pages), _ptr(v_pages), _ptr(k_scales), int(k_pages.shape[0]),
            _ptr(page_table), int(page_table.shape[1]), _ptr(seq_lens), batch, scale, _ptr(out),
            1 if out.dtype == torch.float32 else 0, _ptr(workspace),
            int(workspace.numel() * workspace.element_size()), _stream()), "novakv_decode_attention_scaled")

    def novakv_decode_attention_sink(self, layer, q, k_pages, v_pages, k_scales, sink_logits, page_table, seq_lens,
                                     out, workspace, sm_scale=None):
        """Decode step with a learned sink logit per query head (k_scales may be None)."""
        import torch
        batch = int(q.shape[0])
        scale = float(self.head_dim) ** -0.5 if sm_scale is None else float(sm_scale)
        _check(self.lib, self.lib.novakv_decode_attention_sink(
            self.handle, layer, _ptr(q), _ptr(k_pages), _ptr(v_pages), _ptr(k_scales) if k_scales is not None else None,
            _ptr(sink_logits), int(k_pages.shape[0]), _ptr(page_table), int(page_table.shape[1]), _ptr(seq_lens),
            batch, scale, _ptr(out), 1 if out.dtype == torch.float32 else 0, _ptr(workspace),
            int(workspace.numel() * workspace.element_size()), _stream()), "novakv_decode_attention_sink")

    def novakv_decode_attention_banded(self, layer, q, k_pages, v_pages, k_scales, sink_logits, page_table,
                                       quant_lens, band_k, band_v, n_sink, band_meta, out, workspace, sm_scale=None):
        """Decode step on a cache with a BF16 sink-plus-recent band (band_k/band_v [batch][cap][Hkv][d])."""
        import torch
        batch = int(q.shape[0])
        scale = float(self.head_dim) ** -0.5 if sm_scale is None else float(sm_scale)
        _check(self.lib, self.lib.novakv_decode_attention_banded(
            self.handle, layer, _ptr(q), _ptr(k_pages), _ptr(v_pages),
            _ptr(k_scales) if k_scales is not None else None, _ptr(sink_logits) if sink_logits is not None else None,
            int(k_pages.shape[0]), _ptr(page_table), int(page_table.shape[1]), _ptr(quant_lens), _ptr(band_k),
            _ptr(band_v), int(band_k.shape[1]), int(n_sink), _ptr(band_meta), batch, scale, _ptr(out),
            1 if out.dtype == torch.float32 else 0, _ptr(workspace),
            int(workspace.numel() * workspace.element_size()), _stream()), "novakv_decode_attention_banded")

    def novakv_value_meta_page_bytes(self):
        return int(self.lib.novakv_value_meta_page_bytes(self.handle))

    def novakv_encode_append_deployed(self, layer, k_new, v_new, tok_seq, tok_pos, k_pages, v_pages, k_scales, v_meta,
                                      page_table, seq_lens):
        n_tokens = int(k_new.shape[0]) if k_new is not None else 0
        _check(self.lib, self.lib.novakv_encode_append_deployed(
            self.handle, layer, _ptr(k_new), _ptr(v_new), _ptr(tok_seq), _ptr(tok_pos), n_tokens,
            _ptr(k_pages), _ptr(v_pages), _ptr(k_scales), _ptr(v_meta), int(k_pages.shape[0]), _ptr(page_table),
            int(page_table.shape[1]), int(page_table.shape[0]), _ptr(seq_lens), _stream()),
            "novakv_encode_append_deployed")

    def novakv_band_append_staging_bytes(self, batch, block):
        return int(self.lib.novakv_band_append_staging_bytes(self.handle, int(batch), int(block)))

    def novakv_band_append(self, layer, k_new, v_new, band_k, band_v, n_sink, n_rec, block, band_meta, quant_lens,
                           k_pages, v_pages, k_scales, v_meta, page_table, seq_lens, staging):
        """One new token per sequence into the BF16 band; blocks that leave it are encoded (all on the device)."""
        opt = lambda t: _ptr(t) if t is not None else None
        _check(self.lib, self.lib.novakv_band_append(
            self.handle, layer, _ptr(k_new), _ptr(v_new), int(k_new.shape[0]), _ptr(band_k), _ptr(band_v),
            int(band_k.shape[1]), int(n_sink), int(n_rec), int(block), _ptr(band_meta), _ptr(quant_lens),
            _ptr(k_pages), _ptr(v_pages), opt(k_scales), opt(v_meta), int(k_pages.shape[0]), _ptr(page_table),
            int(page_table.shape[1]), _ptr(seq_lens), _ptr(staging), int(staging.numel() * staging.element_size()),
            _stream()), "novakv_band_append")

    def novakv_decode_attention_deployed(self, layer, q, k_pages, v_pages, k_scales, v_meta, sink_logits, page_table,
                                         quant_lens, band_k, band_v, n_sink, band_meta, out, workspace, sm_scale=None):
        """Decode on the deployed format; band_k = band_v = band_meta = None: no BF16 band."""
        import torch
        batch = int(q.shape[0])
        scale = float(self.head_dim) ** -0.5 if sm_scale is None else float(sm_scale)
        opt = lambda t: _ptr(t) if t is not None else None
        _check(self.lib, self.lib.novakv_decode_attention_deployed(
            self.handle, layer, _ptr(q), _ptr(k_pages), _ptr(v_pages), _ptr(k_scales), _ptr(v_meta), opt(sink_logits),
            int(k_pages.shape[0]), _ptr(page_table), int(page_table.shape[1]), _ptr(quant_lens), opt(band_k),
            opt(band_v), int(band_k.shape[1]) if band_k is not None else 0, int(n_sink), opt(band_meta), batch, scale,
            _ptr(out), 1 if out.dtype == torch.float32 else 0, _ptr(workspace),
            int(workspace.numel() * workspace.element_size()), _stream()), "novakv_decode_attention_deployed")

    def novakv_decode_attention_noalloc(self, layer, q, k_pages, v_pages, page_table, seq_lens, out, sm_scale=None):
        """Decode step whose scratch is the library's fixed device array (no workspace argument)."""
        import torch
        scale = float(self.head_dim) ** -0.5 if sm_scale is None else float(sm_scale)
        _check(self.lib, self.lib.novakv_decode_attention_noalloc(
            self.handle, layer, _ptr(q), _ptr(k_pages), _ptr(v_pages), int(k_pages.shape[0]), _ptr(page_table),
            int(page_table.shape[1]), _ptr(seq_lens), int(q.shape[0]), scale, _ptr(out),
            1 if out.dtype == torch.float32 else 0, _stream()), "novakv_decode_attention_noalloc")

    def novakv_last_device_status(self):
        word = c_uint32(0)
        _check(self.lib, self.lib.novakv_last_device_status(self.handle, _stream(), ctypes.byref(word)),
               "novakv_last_device_status")
        return int(word.value)

    def novakv_step_staging_bytes(self, batch, n_tokens):
        return int(self.lib.novakv_step_staging_bytes(self.handle, batch, n_tokens))

    def novakv_step_host(self, layer, k_new_host, v_new_host, tok_seq_host, tok_pos_host, q_host, k_pages,
                         v_pages, page_table, seq_lens, out_host, staging, workspace, sm_scale=None, wait=True):
        """Host tensors (ideally pinned) in, host tensor out; the cache stays on the device.  wait=False enqueues
        the step without waiting for it (``novakv_step_host_async``): read ``out_host`` after a stream sync."""
        n_tokens = int(k_new_host.shape[0]) if k_new_host is not None else 0
        batch = int(q_host.shape[0])
        scale = float(self.head_dim) ** -0.5 if sm_scale is None else float(sm_scale)
        fn = self.lib.novakv_step_host if wait else self.lib.novakv_step_host_async
        _check(self.lib, fn(
            self.handle, layer, _ptr(k_new_host), _ptr(v_new_host), _ptr(tok_seq_host), _ptr(tok_pos_host),
            n_tokens, _ptr(q_host), _ptr(k_pages), _ptr(v_pages), int(k_pages.shape[0]), _ptr(page_table),
            int(page_table.shape[1]), _ptr(seq_lens), batch, scale, _ptr(out_host), _ptr(staging),
            int(staging.numel() * staging.element_size()), _ptr(workspace),
            int(workspace.numel() * workspace.element_size()), _stream()), "novakv_step_host")

    # -- helpers ----------------------------------------------------------------------------
    def novakv_search_coefficients(self, layer, which, coef, idx_out):
        _check(self.lib, self.lib.novakv_search_coefficients(self.handle, layer, which, _ptr(coef),
                                                             int(coef.shape[0]), _ptr(idx_out), _stream()),
               "novakv_search_coefficients")

    def novakv_bf16_workspace_bytes(self, batch, max_pages_per_seq):
        return int(self.lib.novakv_bf16_workspace_bytes(self.handle, batch, max_pages_per_seq))

    def novakv_bf16_decode_attention(self, q, k_pages_bf16, v_pages_bf16, page_table, seq_lens, out, workspace,
                                     sm_scale=None, window=0):
        import torch
        scale = float(self.head_dim) ** -0.5 if sm_scale is None else float(sm_scale)
        _check(self.lib, self.lib.novakv_bf16_decode_attention(
            self.handle, _ptr(q), _ptr(k_pages_bf16), _ptr(v_pages_bf16), int(k_pages_bf16.shape[0]),
            _ptr(page_table), int(page_table.shape[1]), _ptr(seq_lens), int(q.shape[0]), scale, int(window),
            _ptr(out), 1 if out.dtype == torch.float32 else 0, _ptr(workspace),
            int(workspace.numel() * workspace.element_size()), _stream()), "novakv_bf16_decode_attention")

    def novakv_profile_enable(self, on=True):
        _check(self.lib, self.lib.novakv_profile_enable(self.handle, 1 if on else 0), "novakv_profile_enable")

    def novakv_profile_read(self, kind):
        ms, n = c_double(0), c_long(0)
        _check(self.lib, self.lib.novakv_profile_read(self.handle, kind, ctypes.byref(ms), ctypes.byref(n)),
               "novakv_profile_read")
        return float(ms.value), int(n.value)

    def novakv_debug_set_scan_ctas(self, n_ctas):
        _check(self.lib, self.lib.novakv_debug_set_scan_ctas(self.handle, int(n_ctas)), "novakv_debug_set_scan_ctas")

    def novakv_debug_set_value_path(self, path):
        _check(self.lib, self.lib.novakv_debug_set_value_path(self.handle, int(path)), "novakv_debug_set_value_path")

    def novakv_debug_set_segment_weight(self, pages):
        _check(self.lib, self.lib.novakv_debug_set_segment_weight(self.handle, int(pages)),
               "novakv_debug_set_segment_weight")

    def novakv_debug_set_fused_merge(self, on):
        _check(self.lib, self.lib.novakv_debug_set_fused_merge(self.handle, int(bool(on))), "novakv_debug_set_fused_merge")

    def novakv_launch_count(self):
        return int(self.lib.novakv_launch_count(self.handle))
