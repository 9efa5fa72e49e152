#!/usr/bin/env python
"""Benchmark of the NOVA-KV hot path on B200: one step = append one new token per sequence to
the 2-bit VQ cache (transform + nearest-codeword encode) and one decode-attention pass over it.

Default workload: Qwen3-8B-shaped layer (32 query / 8 KV heads, d = 128), batch 8, S = 16384,
synthetic inputs.  Metric: decode-attention HBM GB/s at 2 bits/element = algorithmic bytes the
decode step must read (packed indices + codebooks + transforms + q/out) / time of the whole step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--no-sweep]

N > 1: one rank per GPU under torch.distributed.run (started by this script itself when it is not
already running under a launcher); every rank runs its own batch (weak scaling, no collective on the
data path), time is the max over ranks.  `--impl reference` times the CPU oracle on the host cores on
a bounded sample of the same workload.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode_attention_hbm_gbps_at_2bit"
UNIT = "GB/s"
NOMINAL_HBM_GBPS = 8000.0
FALLBACK_PEAK_GBPS = 6650.0


def env_rank():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_PEAK_GBPS, "fallback"


def ncu_traffic_per_launch(name):
    """dram bytes per launch of the scan kernel from the committed ncu summary, if there is one."""
    p = os.path.join(ROOT, "profiles", name)
    try:
        for line in open(p):
            if line.startswith("dram_bytes_per_launch:"):
                return float(line.split(":")[1].split()[0])
    except OSError:
        pass
    return None


class ClockSampler:
    """Samples SM clock, power and clock-event reasons through NVML in a thread while the timed
    region runs (read-only queries; no GPU setting is touched)."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, cuda_index, period_s=0.0):
        import threading
        self.samples, self.mask, self.max_mhz, self.err = [], 0, None, None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            p = torch.cuda.get_device_properties(cuda_index)
            try:
                bus = "%08x:%02x:%02x.0" % (p.pci_domain_id, p.pci_bus_id, p.pci_device_id)
                self.h = pynvml.nvmlDeviceGetHandleByPciBusId(bus.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(cuda_index)
            self.nv = pynvml
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as e:          # noqa: BLE001
            self.err = f"nvml unavailable: {e}"
            return

        def loop():
            nv = self.nv
            while not self._stop.is_set():
                try:
                    mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                    pw = nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                    try:
                        m = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                    except Exception:
                        m = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                    self.samples.append((float(mhz), pw))
                    self.mask |= int(m)
                except Exception as e:   # noqa: BLE001
                    self.err = str(e)
                    return
                if period_s > 0:
                    self._stop.wait(period_s)

        self._thread = threading.Thread(target=loop, daemon=True)
        self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "samples": 0, "reasons": [self.err or "no samples"]}
        mhz = sorted(s[0] for s in self.samples)
        return {"sm_mhz": mhz[len(mhz) // 2], "sm_min_mhz": mhz[0], "sm_max_mhz": self.max_mhz,
                "power_w_max": round(max(s[1] for s in self.samples), 1), "samples": len(mhz),
                "reasons": sorted(name for bit, name in self.REASONS.items() if self.mask & bit)}


# ------------------------------------------------------------------------------------------------
def algorithmic_decode_bytes(wl, n_tables_heads=None):
    """Bytes the decode step must move: indices + codebooks (fp32 keys, fp16 values) + the two
    transforms it applies + queries (bf16) + outputs (fp32) + page table and lengths."""
    s = wl.shape
    d, L = s.head_dim, s.head_dim // 4
    idx = wl.decode_index_bytes()
    cb = s.n_kv_heads * L * 256 * 4 * (4 + 2)
    tr = s.n_kv_heads * 2 * d * d * 4
    qo = wl.batch * s.n_q_heads * d * (2 + 4)
    pt = int(np.sum((wl.seq_lens.astype(np.int64) + 63) // 64)) * 4 + wl.batch * 4
    return idx + cb + tr + qo + pt, idx


def fill_cache_gpu(case_ctx, cache, laws, seq_lens, seed, share_content=False):
    """Fill the paged cache with the GPU encoder (the path under test elsewhere)."""
    import torch
    from paper_2608_04074_b200 import synth
    from paper_2608_04074_b200.runtime import bf16_tensor
    cache.seq_lens.zero_()
    CH = 8192
    if not share_content:
        for b, n in enumerate(seq_lens):
            n = int(n)
            for t0 in range(0, n, CH):
                m = min(CH, n - t0)
                k, v = synth.draw_kv(laws, seed + 131 * b + t0 // CH, m)
                cache.append(0, bf16_tensor(k), bf16_tensor(v),
                             torch.full((m,), b, dtype=torch.int32, device="cuda"),
                             torch.arange(t0, t0 + m, dtype=torch.int32, device="cuda"))
        return
    # one drawn sequence, encoded once, its pages copied to every other sequence (distinct physical pages)
    nmax = int(max(seq_lens))
    b0 = int(np.argmax(seq_lens))
    for t0 in range(0, nmax, CH):
        m = min(CH, nmax - t0)
        k, v = synth.draw_kv(laws, seed + t0 // CH, m)
        cache.append(0, bf16_tensor(k), bf16_tensor(v), torch.full((m,), b0, dtype=torch.int32, device="cuda"),
                     torch.arange(t0, t0 + m, dtype=torch.int32, device="cuda"))
    src = cache.page_table[b0].long()
    for b, n in enumerate(seq_lens):
        if b == b0:
            continue
        npg = (int(n) + 63) // 64
        dst = cache.page_table[b, :npg].long()
        cache.k_pages[dst] = cache.k_pages[src[:npg]]
        cache.v_pages[dst] = cache.v_pages[src[:npg]]
        if getattr(cache, "k_scales", None) is not None:
            cache.k_scales[dst] = cache.k_scales[src[:npg]]
    cache.seq_lens.copy_(torch.from_numpy(np.asarray(seq_lens, np.int32)).cuda())


def time_bf16_comparator(ctx, wl, dev, steps, flush):
    """The in-house uncompressed bf16 decode kernel on the same shape (random bf16 cache content)."""
    import torch
    from paper_2608_04074_b200 import synth
    s = wl.shape
    table, n_pages = synth.shuffled_page_table(31, np.maximum(wl.seq_lens, 1), 64)
    kp = torch.empty((n_pages, s.n_kv_heads, 64, s.head_dim), dtype=torch.bfloat16, device=dev).normal_()
    vp = torch.empty((n_pages, s.n_kv_heads, 64, s.head_dim), dtype=torch.bfloat16, device=dev).normal_()
    pt = torch.from_numpy(np.where(table < 0, 0, table).astype(np.int32)).to(dev)
    sl = torch.from_numpy(wl.seq_lens.astype(np.int32)).to(dev)
    q = torch.empty((wl.batch, s.n_q_heads, s.head_dim), dtype=torch.bfloat16, device=dev).normal_()
    out = torch.empty((wl.batch, s.n_q_heads, s.head_dim), dtype=torch.float32, device=dev)
    ws = torch.empty(ctx.novakv_bf16_workspace_bytes(wl.batch, table.shape[1]), dtype=torch.uint8, device=dev)
    tt = time_steps(lambda: ctx.novakv_bf16_decode_attention(q, kp, vp, pt, sl, out, ws), steps, 3, flush)
    ms = statistics.median(tt)
    kv_bytes = int(np.sum(wl.seq_lens.astype(np.int64))) * s.n_kv_heads * 2 * s.head_dim * 2
    del kp, vp
    torch.cuda.empty_cache()
    return {"ms": round(ms, 4), "kv_bytes": kv_bytes, "gbps": round(kv_bytes / (ms * 1e-3) / 1e9, 1)}


def time_steps(fn, steps, warmup, flush, after_warmup=None):
    """Per-step CUDA-event timing on the current stream; the L2 flush sits outside the events."""
    import torch
    for _ in range(warmup):
        flush(); fn()
    torch.cuda.synchronize()
    if after_warmup is not None:
        after_warmup()
    evs = []
    for _ in range(steps):
        flush()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); fn(); b.record()
        evs.append((a, b))
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in evs]


def med_min(times):
    return round(statistics.median(times), 5), round(min(times), 5)


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2608_04074_b200 import synth, workloads
    from paper_2608_04074_b200.binding import Context
    from paper_2608_04074_b200.runtime import PagedCache, bf16_tensor

    rank, local_rank, world = env_rank()
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"

    wl = workloads.qwen3_8b(batch=args.batch, seq_len=args.seq_len, calib_tokens=args.calib_tokens, lloyd_iters=args.lloyd_iters)
    laws = wl.laws()
    cal = wl.calibration(laws)
    s = wl.shape
    ctx = Context(s.n_q_heads, s.n_kv_heads, s.head_dim, device=local_rank)
    ctx.novakv_load_calibration(0, cal)
    B, S = wl.batch, args.seq_len
    cache = PagedCache(ctx, wl.seq_lens, capacity_tokens=wl.seq_lens + 64, seed=17 + rank, device=dev)
    fill_cache_gpu(ctx, cache, laws, wl.seq_lens, seed=5000 + 100000 * rank)

    # a sample of what the GPU encoder stored (the CPU-baseline leg compares it with the oracle's indices)
    parity = None
    if rank == 0:
        from paper_2608_04074_b200 import cache_format
        kp = cache.k_pages.cpu().numpy().reshape(cache.n_pages, s.n_kv_heads, -1)
        vp = cache.v_pages.cpu().numpy().reshape(cache.n_pages, s.n_kv_heads, -1)
        parity = {"samples": []}
        gen = synth.rng(4711)
        for b, chunk in ((0, 1 if S > 8192 else 0), (B - 1, 0)):
            m = min(8192, S - chunk * 8192)
            pick = np.sort(gen.choice(m, size=min(512, m), replace=False))
            kk, vv = synth.draw_kv(laws, 5000 + 100000 * rank + 131 * b + chunk, m)        # what fill_cache_gpu drew
            gk, gv = cache_format.read_tokens(kp, vp, cache.page_table_host[b], s.n_kv_heads, s.head_dim, 0, S)
            parity["samples"].append(dict(k=synth.to_bf16_representable(kk[pick]), v=synth.to_bf16_representable(vv[pick]),
                                          gk=gk[chunk * 8192 + pick], gv=gv[chunk * 8192 + pick]))
        parity["seq0_idx"] = cache_format.read_tokens(kp, vp, cache.page_table_host[0], s.n_kv_heads, s.head_dim, 0, S)
        del kp, vp

    # step inputs: one new token per sequence at position S, one query per sequence
    k1, v1 = synth.draw_kv(laws, 7001 + rank, B)
    q = synth.draw_q(laws, 7002 + rank, B)
    k1d, v1d, qd = bf16_tensor(k1, dev), bf16_tensor(v1, dev), bf16_tensor(q, dev)
    tok_seq = torch.arange(B, dtype=torch.int32, device=dev)
    tok_pos = torch.full((B,), S, dtype=torch.int32, device=dev)
    out = torch.empty((B, s.n_q_heads, s.head_dim), dtype=torch.float32, device=dev)
    flush_buf = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)   # > 126 MB L2

    def flush():
        flush_buf.zero_()

    def step():
        cache.append(0, k1d, v1d, tok_seq, tok_pos)
        cache.decode(0, qd, out=out)

    wl_after = workloads.qwen3_8b(batch=B, seq_len=S + 1)
    alg_bytes, idx_bytes = algorithmic_decode_bytes(wl_after)

    # ---- device-resident timing -------------------------------------------------------------
    ctx.novakv_profile_enable(False)
    if parity is not None:
        cache.decode(0, qd, out=out)          # before any append: attends over the S tokens sampled above
        parity["seq0_out"] = out[0].cpu().numpy()
        parity["seq0_q"] = synth.to_bf16_representable(q[0])
    for _ in range(2):
        step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    # pass A: the timed region proper, K steps, no intra-step events (they cost ~15 % of a 80 us step)
    mark = {}

    def after_warmup():
        mark["launches0"] = ctx.novakv_launch_count()

    times = time_steps(step, args.steps, args.warmup, flush, after_warmup)
    launches = ctx.novakv_launch_count() - mark["launches0"]
    # pass B: the same K steps again with the library's per-kernel events on: scan / append kernel time
    ctx.novakv_profile_enable(True)

    def after_warmup_b():
        ctx.novakv_profile_read(0); ctx.novakv_profile_read(1)

    time_steps(step, args.steps, 3, flush, after_warmup_b)
    s1_ms, s1_n = ctx.novakv_profile_read(0)
    enc_ms, enc_n = ctx.novakv_profile_read(1)
    ctx.novakv_profile_enable(False)
    status = ctx.novakv_last_device_status()
    ms_step = sum(times) / len(times)
    if world > 1:
        t = torch.tensor([ms_step], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_step = float(t.item())

    # ---- decode only / encode only (explanatory numbers) ------------------------------------
    dec_times = time_steps(lambda: cache.decode(0, qd, out=out), args.steps, 3, flush)
    dec_ms, dec_min = med_min(dec_times)
    nowarm = time_steps(lambda: cache.decode(0, qd, out=out), args.steps, 3, lambda: None)
    dec_ms_warm_l2 = statistics.median(nowarm)

    # ---- the CUDA-core value-side variant and the uncompressed bf16 comparator, same shape ------
    ctx.novakv_debug_set_value_path(0)
    cc_times = time_steps(lambda: cache.decode(0, qd, out=out), args.steps, 3, flush)
    ctx.novakv_debug_set_value_path(1)
    cc_ms, cc_min = med_min(cc_times)
    bf16 = time_bf16_comparator(ctx, wl_after, dev, max(5, args.steps // 2), flush)

    # ---- end to end from pinned host buffers through the C ABI --------------------------------
    pin = lambda t: t.cpu().pin_memory()
    k1h, v1h, qh, seqh, posh = pin(k1d), pin(v1d), pin(qd), pin(tok_seq), pin(tok_pos)
    out_h = torch.empty(out.shape, dtype=torch.float32).pin_memory()
    staging = torch.empty(ctx.novakv_step_staging_bytes(B, B), dtype=torch.uint8, device=dev)

    def step_host():
        ctx.novakv_step_host(0, k1h, v1h, seqh, posh, qh, cache.k_pages, cache.v_pages, cache.page_table,
                             cache.seq_lens, out_h, staging, cache.workspace)

    def step_host_async():
        ctx.novakv_step_host(0, k1h, v1h, seqh, posh, qh, cache.k_pages, cache.v_pages, cache.page_table,
                             cache.seq_lens, out_h, staging, cache.workspace, wait=False)

    e2e_times = time_steps(step_host, args.steps, 3, flush)
    # the same step enqueued without the host waiting inside the call: the closing event then sits right behind the
    # kernel that writes the output into the page-locked host buffer, so the interval is the device timeline of the
    # host -> device gather, the append, the decode and the device -> host write, without the host's wake-up
    e2e_dev_times = time_steps(step_host_async, args.steps, 3, flush)
    torch.cuda.synchronize()
    # median: this call returns to Python every step, where the clock-sampling thread of this script holds
    # the interpreter lock for milliseconds now and then; the mean is reported beside it
    e2e_ms = statistics.median(e2e_times)
    e2e_mean_ms = sum(e2e_times) / len(e2e_times)
    # what the same harness measures for a step that launches nothing and only synchronises the stream: the
    # part of the end-to-end time that is neither copy nor kernel (return from the wait, the closing event)
    e2e_floor_ms = statistics.median(time_steps(lambda: torch.cuda.current_stream().synchronize(), args.steps, 3, flush))
    if world > 1:
        t = torch.tensor([e2e_ms], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())
    # the sampler ran from before the warm-up through every timed loop above (NVML queries take
    # milliseconds, so the few-ms headline loop alone would give one sample)
    clocks = sampler.stop() if sampler else None
    h2d = int(k1h.numel() * 2 + v1h.numel() * 2 + qh.numel() * 2 + seqh.numel() * 4 + posh.numel() * 4)
    d2h = int(out_h.numel() * 4)

    result = None
    if rank == 0:
        peak, peak_kind = measured_peak()
        s1_avg_ms = s1_ms / max(s1_n, 1)
        s1_bytes = alg_bytes            # the scan kernel and its two small neighbours move all of it
        achieved = s1_bytes / (s1_avg_ms * 1e-3) / 1e9
        value = alg_bytes * world / (ms_step * 1e-3) / 1e9
        result = {
            "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": round(ms_step, 5), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None,
            "dtype": "f32 accumulation; f32/f16 score-table entries; f16 MMA operands on the value side (7-bit grid codewords)",
            "data": "synthetic", "ms_per_step_min": round(min(times), 5),
            "config": {"workload": f"qwen3_8b_shape decode step: Hq=32 Hkv=8 d=128 B={B} S={S}+1 per GPU, "
                                   "2-bit VQ K and V (g=4, 256-entry codebooks), bf16 q, 64-token pages; "
                                   "step = encode_append of B tokens + decode_attention",
                       "batch_per_gpu": B, "seq_len": S, "l2": "flushed between timed steps (256 MB write)",
                       "parallelism": f"replicas x{world}, no data-path collective"},
            "pct_of_8TBps": round(100 * value / world / NOMINAL_HBM_GBPS, 2),
            "algorithmic_bytes_per_step": alg_bytes, "index_bytes_per_step": idx_bytes,
            "clocks": clocks,
            "e2e": {"value": round(alg_bytes * world / (e2e_ms * 1e-3) / 1e9, 2), "unit": UNIT,
                    "ms_per_step": round(e2e_ms, 5), "ms_per_step_mean": round(e2e_mean_ms, 5),
                    "ms_of_an_empty_step_in_this_harness": round(e2e_floor_ms, 5),
                    "ms_per_step_device_timeline": round(statistics.median(e2e_dev_times), 5),
                    "note": "value and ms_per_step: novakv_step_host returns after the stream wait and the host records "
                            "the closing event afterwards; ms_per_step_device_timeline: novakv_step_host_async, the "
                            "closing event directly behind the kernel that writes the host output",
                    "ms_above_the_device_resident_step": round(e2e_ms - ms_step, 5),
                    "stat": "median of the K per-step times", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": int(launches),
            "roofline": {"kernel": "novakv_decode_stage1_kernel<128,4>", "bound": "hbm",
                         "achieved": round(achieved, 1), "peak": peak, "peak_kind": f"of {peak_kind}",
                         "unit": "GB/s", "frac": round(achieved / peak, 4),
                         "avg_launch_ms": round(s1_avg_ms, 5), "launches_timed": s1_n,
                         "timing": "CUDA events around the kernel, second pass of the same K steps",
                         "traffic": ncu_traffic_per_launch("decode_stage1_qwen3_8b_B8_S16384.md")},
            "decode_only": {"ms": round(dec_ms, 5), "ms_min": dec_min, "gbps": round(alg_bytes / (dec_ms * 1e-3) / 1e9, 1),
                            "pct_of_8TBps": round(100 * alg_bytes / (dec_ms * 1e-3) / 1e9 / NOMINAL_HBM_GBPS, 2),
                            "ms_l2_not_flushed": round(dec_ms_warm_l2, 5)},
            "decode_only_cuda_core_value_side": {"ms": round(cc_ms, 5), "ms_min": cc_min,
                                                 "gbps": round(alg_bytes / (cc_ms * 1e-3) / 1e9, 1),
                                                 "note": "the variant that keeps tensor cores out of the decode path altogether "
                                                         "(north_star's literal reading); the headline runs the value-side "
                                                         "contraction on tensor cores"},
            "bf16_comparator": dict(bf16, speedup_of_2bit_decode=round(bf16["ms"] / dec_ms, 2)),
            "encode_append": {"tokens": B, "avg_kernel_ms": round(enc_ms / max(enc_n, 1), 5)},
            "device_status": status,
        }

    # ---- sweep: long-context bandwidth configs and prefill encode (rank 0 of a 1-GPU run only) ----
    oracle_jobs = []
    if rank == 0 and world == 1 and not args.no_sweep:
        sweep = []
        del cache
        torch.cuda.empty_cache()
        for (b2, s2) in ((64, 32768), (64, 65536)):
            wl2 = workloads.qwen3_8b(batch=b2, seq_len=s2)
            c2 = PagedCache(ctx, wl2.seq_lens, seed=23, device=dev)
            fill_cache_gpu(ctx, c2, laws, wl2.seq_lens, seed=9000, share_content=True)
            q2 = bf16_tensor(synth.draw_q(laws, 7100, b2), dev)
            o2 = torch.empty((b2, s.n_q_heads, s.head_dim), dtype=torch.float32, device=dev)
            ctx.novakv_profile_enable(True); ctx.novakv_profile_read(0)
            tt = time_steps(lambda: c2.decode(0, q2, out=o2), max(5, args.steps // 2), 3, lambda: None)
            k_ms, k_n = ctx.novakv_profile_read(0)
            ctx.novakv_profile_enable(False)
            ab, ib = algorithmic_decode_bytes(wl2)
            ms, ms_min = med_min(tt)
            oracle_jobs.append((f"qwen3_8b_shape B={b2} S={s2}", wl2, laws, cal))
            del c2
            torch.cuda.empty_cache()
            bf = time_bf16_comparator(ctx, wl2, dev, 5, lambda: None)
            sweep.append({"workload": f"qwen3_8b_shape B={b2} S={s2} decode only, inputs larger than L2",
                          "ms": round(ms, 4), "ms_min": round(ms_min, 4), "gbps": round(ab / (ms * 1e-3) / 1e9, 1),
                          "pct_of_8TBps": round(100 * ab / (ms * 1e-3) / 1e9 / NOMINAL_HBM_GBPS, 2),
                          "scan_kernel_ms": round(k_ms / max(k_n, 1), 4),
                          "scan_kernel_frac_of_measured_peak": round(ab / (k_ms / max(k_n, 1) * 1e-3) / 1e9 / measured_peak()[0], 4),
                          "algorithmic_bytes": ab,
                          "bf16_comparator": dict(bf, speedup_of_2bit_decode=round(bf["ms"] / ms, 2))})
            result["roofline"].setdefault("long_context", []).append(
                {"workload": f"B={b2} S={s2}", "achieved": round(ab / (k_ms / max(k_n, 1) * 1e-3) / 1e9, 1),
                 "frac": sweep[-1]["scan_kernel_frac_of_measured_peak"], "avg_launch_ms": sweep[-1]["scan_kernel_ms"]})
            del q2, o2
            torch.cuda.empty_cache()
        # paged serving mix: 128 ragged sequences, append 128 tokens then decode (Qwen3-8B KV shape)
        wl5 = workloads.paged_mix()
        c5 = PagedCache(ctx, wl5.seq_lens, capacity_tokens=wl5.seq_lens + 64, seed=37, device=dev)
        fill_cache_gpu(ctx, c5, laws, wl5.seq_lens, seed=9100, share_content=True)
        n5 = wl5.batch
        k5, v5 = synth.draw_kv(laws, 7300, n5)
        k5d, v5d = bf16_tensor(k5, dev), bf16_tensor(v5, dev)
        q5 = bf16_tensor(synth.draw_q(laws, 7301, n5), dev)
        o5 = torch.empty((n5, s.n_q_heads, s.head_dim), dtype=torch.float32, device=dev)
        seq5 = torch.arange(n5, dtype=torch.int32, device=dev)
        pos5 = torch.from_numpy(wl5.seq_lens.astype(np.int32)).to(dev)

        def step5():
            c5.append(0, k5d, v5d, seq5, pos5)
            c5.decode(0, q5, out=o5)

        tt = time_steps(step5, max(5, args.steps // 2), 3, lambda: None)
        td = time_steps(lambda: c5.decode(0, q5, out=o5), max(5, args.steps // 2), 3, lambda: None)
        wl5b = workloads.paged_mix()
        wl5b.seq_lens = wl5.seq_lens + 1
        ab5, _ = algorithmic_decode_bytes(wl5b)
        ms5, msd5 = statistics.median(tt), statistics.median(td)
        oracle_jobs.append((f"paged mix, {n5} sequences", wl5b, laws, cal))
        sweep.append({"workload": f"paged mix: {n5} sequences, lognormal lengths {int(wl5.seq_lens.min())}..{int(wl5.seq_lens.max())} "
                                  f"(sum {int(wl5.seq_lens.sum())}), 64-token pages shuffled; step = append {n5} tokens + decode",
                      "ms": round(ms5, 4), "decode_only_ms": round(msd5, 4),
                      "gbps": round(ab5 / (ms5 * 1e-3) / 1e9, 1), "decode_only_gbps": round(ab5 / (msd5 * 1e-3) / 1e9, 1),
                      "pct_of_8TBps_decode_only": round(100 * ab5 / (msd5 * 1e-3) / 1e9 / NOMINAL_HBM_GBPS, 2),
                      "algorithmic_bytes": ab5, "device_status": ctx.novakv_last_device_status()})
        del c5
        torch.cuda.empty_cache()
        # prefill encode: 32768 tokens x 8 KV heads x d=128, K and V
        T = 32768
        wl3 = workloads.qwen3_8b(batch=1, seq_len=T)
        c3 = PagedCache(ctx, wl3.seq_lens, seed=29, device=dev)
        kk, vv = synth.draw_kv(laws, 7200, T)
        kd, vd = bf16_tensor(kk, dev), bf16_tensor(vv, dev)
        ts = torch.zeros(T, dtype=torch.int32, device=dev)
        tp = torch.arange(T, dtype=torch.int32, device=dev)
        tt = time_steps(lambda: c3.append(0, kd, vd, ts, tp), 5, 2, lambda: None)
        ms = statistics.median(tt)
        sweep.append({"workload": f"prefill encode {T} tokens x 8 KV heads x d=128 (K and V)", "ms": round(ms, 4),
                      "tokens_per_s": round(T / (ms * 1e-3), 1)})
        # key format with a per-token bf16 scale (2.125 bits per key element): prefill encode, append, decode
        # (its own context: key codebooks trained on normalised coefficients, as the format prescribes)
        cal_s = wl.calibration(laws, key_scale=True)
        ctx_s = Context(s.n_q_heads, s.n_kv_heads, s.head_dim, device=local_rank)
        ctx_s.novakv_load_calibration(0, cal_s)
        c3s = PagedCache(ctx_s, wl3.seq_lens, seed=29, device=dev, key_scale=True)
        tt = time_steps(lambda: c3s.append(0, kd, vd, ts, tp), 5, 2, lambda: None)
        ms_enc_s = statistics.median(tt)
        del c3s, c3
        torch.cuda.empty_cache()
        b6, s6 = 64, 32768
        wl6 = workloads.qwen3_8b(batch=b6, seq_len=s6)
        c6 = PagedCache(ctx_s, wl6.seq_lens, capacity_tokens=wl6.seq_lens + 64, seed=41, device=dev, key_scale=True)
        fill_cache_gpu(ctx_s, c6, laws, wl6.seq_lens, seed=9200, share_content=True)
        q6 = bf16_tensor(synth.draw_q(laws, 7400, b6), dev)
        o6 = torch.empty((b6, s.n_q_heads, s.head_dim), dtype=torch.float32, device=dev)
        td6 = time_steps(lambda: c6.decode(0, q6, out=o6), max(5, args.steps // 2), 3, lambda: None)
        k6, v6 = synth.draw_kv(laws, 7401, b6)
        k6d, v6d = bf16_tensor(k6, dev), bf16_tensor(v6, dev)
        seq6 = torch.arange(b6, dtype=torch.int32, device=dev)
        pos6 = torch.from_numpy(wl6.seq_lens.astype(np.int32)).to(dev)
        ta6 = time_steps(lambda: c6.append(0, k6d, v6d, seq6, pos6), max(5, args.steps // 2), 3, lambda: None)
        ab6, ib6 = algorithmic_decode_bytes(wl6)
        ab6 += int(wl6.seq_lens.astype(np.int64).sum()) * s.n_kv_heads * 2          # the scales are read too
        ms6 = statistics.median(td6)
        sweep.append({"workload": f"scaled key format (bf16 scale per token and KV head, 2.125 bit per key element), qwen3_8b_shape "
                                  f"B={b6} S={s6}: decode only; append of {b6} tokens; prefill encode of {T} tokens "
                                  "(key codebooks trained on normalised coefficients)",
                      "ms": round(ms6, 4), "gbps": round(ab6 / (ms6 * 1e-3) / 1e9, 1),
                      "pct_of_8TBps": round(100 * ab6 / (ms6 * 1e-3) / 1e9 / NOMINAL_HBM_GBPS, 2),
                      "algorithmic_bytes": ab6, "append_ms": round(statistics.median(ta6), 4),
                      "prefill_encode_ms": round(ms_enc_s, 4), "prefill_tokens_per_s": round(T / (ms_enc_s * 1e-3), 1),
                      "device_status": ctx_s.novakv_last_device_status()})
        del c6, q6, o6
        torch.cuda.empty_cache()
        # BF16 sink-plus-recent band (64 + 256 tokens in bf16, the rest in the index cache), primary key format
        from paper_2608_04074_b200.runtime import BandedCache
        c7 = BandedCache(ctx, b6, s6 + 64, n_sink=64, n_rec=256, block=8, seed=43, device=dev)
        fill_cache_gpu(ctx, c7.paged, laws, wl6.seq_lens, seed=9300, share_content=True)
        c7.total[:] = s6
        c7.quant[:] = s6 - 64 - 256
        c7.ring_len[:] = 256
        # band content: synthetic tokens of the workload's law (the same 320 for every sequence)
        kb7, vb7 = synth.draw_kv(laws, 7450, 320)
        c7.band_k[:, :320] = bf16_tensor(kb7, dev)[None]
        c7.band_v[:, :320] = bf16_tensor(vb7, dev)[None]
        c7._sync_meta()
        q7 = bf16_tensor(synth.draw_q(laws, 7500, b6), dev)
        o7 = torch.empty((b6, s.n_q_heads, s.head_dim), dtype=torch.float32, device=dev)
        td7 = time_steps(lambda: c7.decode(0, q7, out=o7), max(5, args.steps // 2), 3, lambda: None)
        ms7 = statistics.median(td7)
        ab7 = ab6 - int(wl6.seq_lens.astype(np.int64).sum()) * s.n_kv_heads * 2            # no scales here
        ab7 += b6 * s.n_kv_heads * 320 * (2 * s.head_dim * 2 - 2 * (s.head_dim // 4))          # 320 tokens in bf16 instead of indices
        # write side: 24 single-token steps through novakv_band_append (new tokens of the workload's law); every
        # 8th step all sequences pass their 8 oldest ring tokens to the encoder (the sequences are aligned)
        kn7, vn7 = synth.draw_kv(laws, 7451, 24 * b6)
        kn7d = bf16_tensor(kn7, dev).reshape(24, b6, s.n_kv_heads, s.head_dim)
        vn7d = bf16_tensor(vn7, dev).reshape(24, b6, s.n_kv_heads, s.head_dim)
        ev7 = []
        for t7 in range(24):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); c7.append_step(0, kn7d[t7], vn7d[t7], mirror=False); e1.record()
            ev7.append((e0, e1))
        torch.cuda.synchronize()
        t7s = [a_.elapsed_time(b_) for a_, b_ in ev7]
        flush7 = [t7s[i] for i in range(8, 24) if i % 8 == 7]
        plain7 = [t7s[i] for i in range(8, 24) if i % 8 != 7]
        c7.refresh_host_state()
        meta7, quant7 = c7.device_state()
        band_state_ok = bool((quant7 == s6 - 320 + 24).all() and (meta7[:, 2] == 256).all())
        sweep.append({"workload": f"BF16 sink-plus-recent band (64 + 256 tokens exact, deferred quantisation in blocks of 8), "
                                  f"qwen3_8b_shape B={b6} S={s6}: decode only; band tokens drawn from the workload's law; "
                                  f"write side = novakv_band_append of {b6} tokens per step",
                      "ms": round(ms7, 4), "gbps": round(ab7 / (ms7 * 1e-3) / 1e9, 1),
                      "pct_of_8TBps": round(100 * ab7 / (ms7 * 1e-3) / 1e9 / NOMINAL_HBM_GBPS, 2),
                      "algorithmic_bytes": ab7,
                      "band_append_ms": round(statistics.median(plain7), 4),
                      "band_append_ms_when_all_sequences_flush_8_tokens": round(statistics.median(flush7), 4),
                      "band_state_after_24_steps_ok": band_state_ok,
                      "device_status": ctx.novakv_last_device_status()})
        del c7, q7, o7
        torch.cuda.empty_cache()
        # the paper's deployed format end to end: scaled VQ keys (2.125 bit) + scalar INT2 values (2.25 bit) + BF16 band
        c8 = BandedCache(ctx_s, b6, s6 + 64, n_sink=64, n_rec=256, block=8, seed=47, device=dev, key_scale=True, int2_values=True)
        fill_cache_gpu(ctx_s, c8.paged, laws, wl6.seq_lens, seed=9400, share_content=True)
        src8 = c8.paged.page_table[int(np.argmax(wl6.seq_lens))].long()
        for bb in range(b6):
            dst8 = c8.paged.page_table[bb].long()
            c8.paged.v_meta[dst8] = c8.paged.v_meta[src8]
        c8.total[:] = s6
        c8.quant[:] = s6 - 64 - 256
        c8.ring_len[:] = 256
        c8.band_k[:, :320] = bf16_tensor(kb7, dev)[None]
        c8.band_v[:, :320] = bf16_tensor(vb7, dev)[None]
        c8._sync_meta()
        q8 = bf16_tensor(synth.draw_q(laws, 7600, b6), dev)
        o8 = torch.empty((b6, s.n_q_heads, s.head_dim), dtype=torch.float32, device=dev)
        td8 = time_steps(lambda: c8.decode(0, q8, out=o8), max(5, args.steps // 2), 3, lambda: None)
        ms8 = statistics.median(td8)
        ab8 = ab7 + int(wl6.seq_lens.astype(np.int64).sum() - 320 * b6) * s.n_kv_heads * (2 + 4)    # key scale + value (scale, zero)
        c8p = PagedCache(ctx_s, wl3.seq_lens, seed=29, device=dev, key_scale=True, int2_values=True)
        tt = time_steps(lambda: c8p.append(0, kd, vd, ts, tp), 5, 2, lambda: None)
        ms_enc8 = statistics.median(tt)
        sweep.append({"workload": f"deployed format of the paper (scaled VQ keys 2.125 bit, scalar INT2 values 2.25 bit, BF16 band 64 + 256), "
                                  f"qwen3_8b_shape B={b6} S={s6}: decode only; prefill encode of {T} tokens "
                                  "(band tokens drawn from the workload's law, key codebooks trained on normalised coefficients)",
                      "ms": round(ms8, 4), "gbps": round(ab8 / (ms8 * 1e-3) / 1e9, 1),
                      "pct_of_8TBps": round(100 * ab8 / (ms8 * 1e-3) / 1e9 / NOMINAL_HBM_GBPS, 2),
                      "algorithmic_bytes": ab8, "prefill_encode_ms": round(ms_enc8, 4),
                      "prefill_tokens_per_s": round(T / (ms_enc8 * 1e-3), 1),
                      "device_status": ctx_s.novakv_last_device_status()})
        del c8, c8p, q8, o8, ctx_s
        torch.cuda.empty_cache()
        # GPT-OSS-20B-shaped hybrid pair: full-attention layer on the 2-bit cache + sliding-window (128) layer in bf16
        wl4 = workloads.gpt_oss_20b(batch=16, seq_len=65536)
        laws4 = wl4.laws()
        cal4 = wl4.calibration(laws4)
        s4 = wl4.shape
        ctx4 = Context(s4.n_q_heads, s4.n_kv_heads, s4.head_dim, device=local_rank)
        ctx4.novakv_load_calibration(0, cal4)
        c4 = PagedCache(ctx4, wl4.seq_lens, seed=41, device=dev)
        fill_cache_gpu(ctx4, c4, laws4, wl4.seq_lens, seed=9200, share_content=True)
        q4 = bf16_tensor(synth.draw_q(laws4, 7400, wl4.batch), dev)
        o4 = torch.empty((wl4.batch, s4.n_q_heads, s4.head_dim), dtype=torch.float32, device=dev)
        tt = time_steps(lambda: c4.decode(0, q4, out=o4), max(5, args.steps // 2), 3, lambda: None)
        ab4, _ = algorithmic_decode_bytes(wl4)
        ms4 = statistics.median(tt)
        oracle_jobs.append(("gpt_oss_20b_shape B=16 S=65536", wl4, laws4, cal4))
        del c4
        torch.cuda.empty_cache()
        bf4 = time_bf16_comparator(ctx4, wl4, dev, 5, lambda: None)
        # the sliding-window layer of the pair stays bf16 (window 128): same comparator kernel, windowed
        table4, n_pages4 = synth.shuffled_page_table(43, wl4.seq_lens, 64)
        kp4 = torch.empty((n_pages4, s4.n_kv_heads, 64, s4.head_dim), dtype=torch.bfloat16, device=dev).normal_()
        vp4 = torch.empty_like(kp4).normal_()
        pt4 = torch.from_numpy(table4.astype(np.int32)).to(dev)
        sl4 = torch.from_numpy(wl4.seq_lens.astype(np.int32)).to(dev)
        ws4 = torch.empty(ctx4.novakv_bf16_workspace_bytes(wl4.batch, table4.shape[1]), dtype=torch.uint8, device=dev)
        tw = time_steps(lambda: ctx4.novakv_bf16_decode_attention(q4, kp4, vp4, pt4, sl4, o4, ws4, window=128), 10, 3, lambda: None)
        sweep.append({"workload": "gpt_oss_20b_shape Hq=64 Hkv=8 d=64 B=16 S=65536: full-attention layer on the 2-bit cache",
                      "ms": round(ms4, 4), "gbps": round(ab4 / (ms4 * 1e-3) / 1e9, 1),
                      "pct_of_8TBps": round(100 * ab4 / (ms4 * 1e-3) / 1e9 / NOMINAL_HBM_GBPS, 2), "algorithmic_bytes": ab4,
                      "bf16_comparator": dict(bf4, speedup_of_2bit_decode=round(bf4["ms"] / ms4, 2)),
                      "sliding_window_128_layer_bf16_ms": round(statistics.median(tw), 4),
                      "device_status": ctx4.novakv_last_device_status()})
        del kp4, vp4
        ctx4.close()
        result["sweep"] = sweep

    if rank == 0:
        result["cpu_baseline"] = cpu_baseline_sample(wl, laws, cal, args, parity, oracle_jobs)
        print(json.dumps(result))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------
def oracle_sample_inputs(wl, laws, cal, n_seq):
    """A bounded sample of the workload for the CPU oracle: n_seq sequences of the full length whose
    indices are 2048 oracle-encoded tokens tiled along the sequence (content does not change timing)."""
    from oracle import novakv_oracle as O
    from paper_2608_04074_b200 import synth
    orc = O.Oracle.from_calibration(cal)
    S = int(wl.seq_lens[0])
    k, v = synth.draw_kv(laws, 8101, 2048)
    k, v = synth.to_bf16_representable(k), synth.to_bf16_representable(v)
    enc = orc.encode(k.astype(np.float64), v.astype(np.float64), with_gaps=False)
    reps = (S + 2047) // 2048
    kidx = np.tile(enc["kidx"], (reps, 1, 1))[:S]
    vidx = np.tile(enc["vidx"], (reps, 1, 1))[:S]
    q = synth.to_bf16_representable(synth.draw_q(laws, 8102, n_seq))
    k1, v1 = synth.draw_kv(laws, 8103, n_seq)
    return orc, kidx, vidx, q, synth.to_bf16_representable(k1), synth.to_bf16_representable(v1)


def oracle_step(orc, kidx, vidx, q, k1, v1):
    """One oracle step on the sample: encode the new tokens, then decode every sampled sequence."""
    orc.encode(k1.astype(np.float64), v1.astype(np.float64), with_gaps=False)
    for b in range(q.shape[0]):
        orc.decode(q[b].astype(np.float64), kidx, vidx)


def _omp_set_threads(n):
    """Thread count of the oracle's OpenMP loops (libgomp runtime call); returns True if it could be set."""
    import ctypes
    try:
        ctypes.CDLL("libgomp.so.1").omp_set_num_threads(int(n))
        return True
    except OSError:
        return False


def oracle_subset(label, wl, laws, cal):
    """Oracle decode time on a stated subset of a sweep workload (first, last and two seeded random sequences,
    all heads), extrapolated linearly in tokens to the whole workload."""
    from oracle import novakv_oracle as O
    from paper_2608_04074_b200 import synth
    orc = O.Oracle.from_calibration(cal)
    n = wl.batch
    pick = sorted(set([0, n - 1] + [int(x) for x in synth.rng(99).choice(n, size=min(2, n), replace=False)]))
    k, v = synth.draw_kv(laws, 8201, 2048)
    enc = orc.encode(synth.to_bf16_representable(k).astype(np.float64), synth.to_bf16_representable(v).astype(np.float64),
                     with_gaps=False)
    q = synth.to_bf16_representable(synth.draw_q(laws, 8202, len(pick)))
    t0 = time.perf_counter()
    for i, b in enumerate(pick):
        S = int(wl.seq_lens[b])
        reps = (S + 2047) // 2048
        orc.decode(q[i].astype(np.float64), np.tile(enc["kidx"], (reps, 1, 1))[:S], np.tile(enc["vidx"], (reps, 1, 1))[:S])
    dt = time.perf_counter() - t0
    sub_tokens = int(sum(int(wl.seq_lens[b]) for b in pick))
    all_tokens = int(wl.seq_lens.astype(np.int64).sum())
    per_tok_bytes = wl.shape.n_kv_heads * 2 * (wl.shape.head_dim // 4)
    return {"workload": label, "sequences": pick, "tokens": sub_tokens, "seconds": round(dt, 3),
            "gbps": round(sub_tokens * per_tok_bytes / dt / 1e9, 6),
            "extrapolated_seconds_whole_workload": round(dt * all_tokens / max(sub_tokens, 1), 2),
            "note": "decode only; time extrapolated linearly in tokens (labelled, not measured)"}


def cpu_baseline_sample(wl, laws, cal, args, parity=None, jobs=()):
    """The CPU-baseline leg: times the oracle on a bounded sample of the benchmark workload (all host cores and one
    thread), on stated subsets of the sweep workloads, and compares what the GPU stored / produced on a sample of
    the benchmark cache with the oracle (index mismatches against the float64 nearest codeword, near-ties)."""
    from oracle import novakv_oracle as O
    n_seq = min(wl.batch, 8)          # about 20 core-seconds of oracle work on the benchmark shape
    orc, kidx, vidx, q, k1, v1 = oracle_sample_inputs(wl, laws, cal, n_seq)
    t0 = time.perf_counter()
    oracle_step(orc, kidx, vidx, q, k1, v1)
    dt = time.perf_counter() - t0
    s = wl.shape
    per_seq_bytes = int(wl.seq_lens[0]) * s.n_kv_heads * 2 * (s.head_dim // 4)
    res = {"value": round(n_seq * per_seq_bytes / dt / 1e9, 6), "unit": UNIT, "cores": O.cpu_threads(), "kind": "oracle",
           "seconds": round(dt, 3),
           "sample": f"{n_seq} of {wl.batch} sequences (S={int(wl.seq_lens[0])}, all heads): oracle encode of "
                     f"{n_seq} new tokens + explicit-dequantise decode; index bytes of the sample / wall time"}
    if _omp_set_threads(1):
        t0 = time.perf_counter()
        oracle_step(orc, kidx, vidx, q[:1], k1[:1], v1[:1])
        dt1 = time.perf_counter() - t0
        _omp_set_threads(O.cpu_threads())
        res["single_thread"] = {"value": round(per_seq_bytes / dt1 / 1e9, 6), "unit": UNIT, "seconds": round(dt1, 3),
                                "sample": "1 sequence of the same workload, one thread"}
    if jobs:
        res["sweep_subsets"] = [oracle_subset(*j) for j in jobs]
    if parity is not None:
        n_groups = mism = near = bad = 0
        max_gap = 0.0
        for smp in parity["samples"]:
            enc = orc.encode(smp["k"].astype(np.float64), smp["v"].astype(np.float64))
            for side, got in (("k", smp["gk"]), ("v", smp["gv"])):
                diff = got != enc[side + "idx"]
                gap = enc[side + "gap"]
                n_groups += int(diff.size)
                mism += int(diff.sum())
                near += int((gap <= 1e-6).sum())
                bad += int((diff & (gap > 1e-6)).sum())
                if diff.any():
                    max_gap = max(max_gap, float(gap[diff].max()))
        gk, gv = parity["seq0_idx"]
        ref = orc.decode(parity["seq0_q"].astype(np.float64), gk, gv)
        err = float(np.abs(parity["seq0_out"] - ref).max() / np.abs(ref).max())
        res["parity_on_benchmark_cache"] = {
            "groups_compared": n_groups, "index_mismatch_vs_f64": mism, "near_ties_le_1e-6": near,
            "index_mismatch_outside_near_ties": bad, "max_gap_among_mismatches": max_gap,
            "decode_max_abs_err_over_out_inf_norm_seq0": round(err, 7), "decode_tolerance": 2e-3,
            "sample": "2 x 512 tokens of the GPU-encoded benchmark cache (all heads, K and V) against the oracle's float64 "
                      "nearest codeword; GPU output of sequence 0 against the oracle's decode of the stored indices"}
    return res


def run_reference(args):
    rank, _, world = env_rank()
    if world > 1:
        # rank 0 alone runs and prints; the others only join the rendezvous (CPU: gloo) and leave
        import torch.distributed as dist
        dist.init_process_group("gloo")
        if rank != 0:
            dist.barrier()
            dist.destroy_process_group()
            return
    _run_reference_rank0(args, world)
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


def _run_reference_rank0(args, world):
    if world > 1:
        # a launcher pins every rank to one OpenMP thread; this rank is the only one that works
        os.environ["OMP_NUM_THREADS"] = str(len(os.sched_getaffinity(0)))
    from oracle import novakv_oracle as O
    from paper_2608_04074_b200 import workloads
    wl = workloads.qwen3_8b(batch=args.batch, seq_len=args.seq_len, calib_tokens=args.calib_tokens, lloyd_iters=args.lloyd_iters)
    laws = wl.laws()
    cal = wl.calibration(laws)
    n_seq = 1
    orc, kidx, vidx, q, k1, v1 = oracle_sample_inputs(wl, laws, cal, n_seq)
    for _ in range(min(args.warmup, 1)):
        oracle_step(orc, kidx, vidx, q, k1, v1)
    steps = max(1, min(args.steps, 5))
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_step(orc, kidx, vidx, q, k1, v1)
    dt = (time.perf_counter() - t0) / steps
    s = wl.shape
    sample_bytes = n_seq * int(wl.seq_lens[0]) * s.n_kv_heads * 2 * (s.head_dim // 4)
    val = round(sample_bytes / dt / 1e9, 6)
    sample = (f"each step: {n_seq} of {wl.batch} sequences (S={int(wl.seq_lens[0])}, all heads), oracle encode + "
              f"decode; {steps} steps timed")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": world, "steps": steps,
        "warmup": min(args.warmup, 1), "ms_per_step": round(dt * 1e3, 3), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"qwen3_8b_shape decode step: Hq=32 Hkv=8 d=128 B={args.batch} S={args.seq_len}, "
                               "CPU oracle on a bounded sample"},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": O.cpu_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_profile_case(args):
    """`--profile-case NAME`: a short decode-only (or encode-only) loop of one workload shape, for profiler captures
    of the kernels the sweep times (the captures summarised under profiles/ were taken with these commands).
    Index bytes are random (timing and counters do not depend on them); prints a small JSON line, not the
    benchmark contract."""
    import torch
    from paper_2608_04074_b200 import synth, workloads
    from paper_2608_04074_b200.binding import Context
    from paper_2608_04074_b200.runtime import PagedCache, bf16_tensor
    name = args.profile_case
    if name == "gptoss":
        wl = workloads.gpt_oss_20b(batch=args.batch, seq_len=args.seq_len, calib_tokens=2048, lloyd_iters=2)
    elif name == "mix":
        wl = workloads.paged_mix(calib_tokens=2048, lloyd_iters=2)
    elif name in ("qwen", "encode", "append"):
        wl = workloads.qwen3_8b(batch=args.batch, seq_len=args.seq_len, calib_tokens=2048, lloyd_iters=2)
    else:
        raise SystemExit(f"unknown profile case {name}")
    laws = wl.laws()
    cal = wl.calibration(laws)
    s = wl.shape
    ctx = Context(s.n_q_heads, s.n_kv_heads, s.head_dim)
    ctx.novakv_load_calibration(0, cal)
    cache = PagedCache(ctx, wl.seq_lens, capacity_tokens=wl.seq_lens + 1 if name == "append" else None, seed=3)
    times = []
    if name == "append":
        # one new token per sequence at the end of its context (the append of a decode step)
        k, v = synth.draw_kv(laws, 7300, wl.batch)
        kd, vd = bf16_tensor(k), bf16_tensor(v)
        ts = torch.arange(wl.batch, dtype=torch.int32, device="cuda")
        tp = torch.from_numpy(wl.seq_lens.astype(np.int32)).cuda()
        fn = lambda: cache.append(0, kd, vd, ts, tp)
    elif name == "encode":
        T = int(wl.seq_lens.sum())
        k, v = synth.draw_kv(laws, 7200, T)
        kd, vd = bf16_tensor(k), bf16_tensor(v)
        ts = torch.repeat_interleave(torch.arange(wl.batch, dtype=torch.int32, device="cuda"),
                                     torch.from_numpy(wl.seq_lens.astype(np.int64)).cuda())
        tp = torch.cat([torch.arange(int(n), dtype=torch.int32, device="cuda") for n in wl.seq_lens])
        fn = lambda: cache.append(0, kd, vd, ts, tp)
    else:
        cache.k_pages.random_(0, 256)
        cache.v_pages.random_(0, 256)
        q = bf16_tensor(synth.draw_q(laws, 5, wl.batch))
        out = torch.empty((wl.batch, s.n_q_heads, s.head_dim), dtype=torch.float32, device="cuda")
        fn = lambda: cache.decode(0, q, out=out)
    times = time_steps(fn, args.steps, args.warmup, lambda: None)
    print(json.dumps({"profile_case": name, "batch": wl.batch, "tokens": int(wl.seq_lens.astype(np.int64).sum()),
                      "ms_median": round(statistics.median(times), 5), "device_status": ctx.novakv_last_device_status()}))


def launch_ranks(n):
    """`--gpus N` outside a launcher: re-run this script as N ranks of one node under torch.distributed.run
    (one rank per GPU, rendezvous on 127.0.0.1) and return its exit code.  NCCL's communicator log is kept
    (in a file per rank, so that standard output stays the one JSON line)."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")
    env.setdefault("NCCL_DEBUG_FILE", os.path.join(os.environ.get("TMPDIR", "/tmp"), "novakv_bench_nccl.%h.%p.log"))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.run(cmd, env=env).returncode


def main():
    sys.setswitchinterval(1e-4)          # let the clock-sampling thread run between short GPU calls
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=8)
    ap.add_argument("--seq-len", type=int, default=16384)
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--profile-case", default=None, choices=["qwen", "gptoss", "mix", "encode", "append"],
                    help="profiling helper: short decode-only (encode-only) loop of one workload shape")
    ap.add_argument("--calib-tokens", type=int, default=8192, help="calibration tokens per KV head (set-up cost only)")
    ap.add_argument("--lloyd-iters", type=int, default=12, help="Lloyd iterations of the calibration (set-up cost only)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.profile_case:
        run_profile_case(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(launch_ranks(args.gpus))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
