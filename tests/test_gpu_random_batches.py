"""GPU parity on seeded random batches: shapes, formats, sink, work-split settings and ragged lengths drawn at
random (fixed seed), every sequence compared with the oracle within the stated output tolerance."""
import numpy as np
import pytest

from gpu_common import Case, check_indices, check_output
from paper_2608_04074_b200 import cache_format, synth, workloads

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    return (t.to(dtype) if dtype is not None else t).cuda()


def test_random_batches_formats_and_split_settings():
    from paper_2608_04074_b200.runtime import PagedCache
    cases = {}

    def get(shape, scaled):
        if (shape, scaled) not in cases:
            wl = (workloads.qwen3_8b(batch=2, seq_len=512, calib_tokens=2048, lloyd_iters=3) if shape == "qwen"
                  else workloads.gpt_oss_20b(batch=2, seq_len=512, calib_tokens=2048, lloyd_iters=3))
            cases[(shape, scaled)] = Case(wl, key_scale=scaled)
        return cases[(shape, scaled)]

    gen = np.random.Generator(np.random.PCG64(2024))
    worst = {}
    for it in range(28):
        shape = "qwen" if gen.random() < 0.5 else "gptoss"
        fmt = int(gen.integers(0, 3))                      # 0: 2-bit K and V, 1: scaled keys, 2: scaled keys + INT2 values
        case = get(shape, fmt > 0)
        batch = int(gen.integers(1, 30))
        lens = gen.integers(0, 700, size=batch).astype(np.int32)
        if gen.random() < 0.3:
            lens[gen.integers(0, batch)] = int(gen.integers(1500, 4000))
        cache = PagedCache(case.ctx, lens, seed=int(gen.integers(0, 1000)), key_scale=fmt == 1, int2_values=fmt == 2)
        encs = []
        for b, n in enumerate(lens):
            if n == 0:
                encs.append(None)
                continue
            k, v, _ = case.draw(5000 + 37 * it + b, int(n), 1)
            k64, v64 = k.astype(np.float64), v.astype(np.float64)
            if fmt == 0:
                e = case.oracle.encode(k64, v64, with_gaps=False)
                cache.store_logical(b, 0, e["kidx"], e["vidx"])
                encs.append((e,))
            else:
                e = case.oracle.encode_scaled(k64, v64, with_gaps=False)
                cache.store_scales(b, 0, e["kscale"])
                if fmt == 1:
                    cache.store_logical(b, 0, e["kidx"], e["vidx"])
                    encs.append((e,))
                else:
                    codes, meta = case.oracle.encode_values_int2(v64)
                    cache.store_logical(b, 0, e["kidx"], cache_format.pack_int2(codes))
                    cache.store_value_meta(b, 0, meta)
                    encs.append((e, codes, meta))
        _, _, q = case.draw(9000 + it, 1, batch)
        use_sink = gen.random() < 0.4
        sink = gen.uniform(-4, 6, size=case.ctx.n_q_heads).astype(np.float32)
        sink64 = sink.astype(np.float64)
        case.ctx.novakv_debug_set_segment_weight(int(gen.choice([0, 3, 24, 100])))
        case.ctx.novakv_debug_set_scan_ctas(int(gen.choice([0, 0, 1, 3, 37])))
        try:
            out = cache.decode(0, _dev(q, torch.bfloat16), sink_logits=_dev(sink) if use_sink else None).cpu().numpy()
            assert case.ctx.novakv_last_device_status() == 0
        finally:
            case.ctx.novakv_debug_set_segment_weight(24)
            case.ctx.novakv_debug_set_scan_ctas(0)
        for b, n in enumerate(lens):
            if n == 0:
                assert not out[b].any()
                continue
            qq = q[b].astype(np.float64)
            e = encs[b][0]
            if fmt == 0:
                ref = (case.oracle.decode_sink(qq, e["kidx"], e["vidx"], sink64) if use_sink
                       else case.oracle.decode(qq, e["kidx"], e["vidx"]))
            elif fmt == 1:
                ref = (case.oracle.decode_sink(qq, e["kidx"], e["vidx"], sink64, kscale=e["kscale"]) if use_sink
                       else case.oracle.decode_scaled(qq, e["kidx"], e["vidx"], e["kscale"]))
            else:
                ref = case.oracle.decode_deployed(qq, e["kidx"], e["kscale"], encs[b][1], encs[b][2],
                                                  sink=sink64 if use_sink else None)
            r = check_output(out[b], ref)
            worst[(shape, fmt)] = max(worst.get((shape, fmt), 0.0), r)
    print({k: f"{v:.2e}" for k, v in sorted(worst.items())})
    assert len(worst) >= 5            # most (shape, format) combinations were drawn


def test_random_appends_formats_and_page_layouts():
    """Appends of 1 .. 700 tokens spread at random over up to 11 sequences with random existing lengths, in a
    random order, in all three formats: indices (near-ties counted), INT2 bytes, scales and (scale, zero)."""
    from paper_2608_04074_b200.runtime import PagedCache
    cases = {}

    def get(shape, scaled):
        if (shape, scaled) not in cases:
            wl = (workloads.qwen3_8b(batch=2, seq_len=512, calib_tokens=2048, lloyd_iters=3) if shape == "qwen"
                  else workloads.gpt_oss_20b(batch=2, seq_len=512, calib_tokens=2048, lloyd_iters=3))
            cases[(shape, scaled)] = Case(wl, key_scale=scaled)
        return cases[(shape, scaled)]

    gen = np.random.Generator(np.random.PCG64(77))
    for it in range(24):
        shape = "qwen" if gen.random() < 0.5 else "gptoss"
        fmt = int(gen.integers(0, 3))
        case = get(shape, fmt > 0)
        nseq = int(gen.integers(1, 12))
        lens0 = gen.integers(0, 200, size=nseq).astype(np.int32)
        n = int(gen.choice([1, 2, 3, 7, 8, 9, 31, 32, 33, 63, 64, 65, 100, 255, 256, 257, 300, 700]))
        cnt = gen.multinomial(n, np.ones(nseq) / nseq).astype(np.int32)
        cache = PagedCache(case.ctx, lens0, capacity_tokens=lens0 + cnt + 1, seed=int(gen.integers(0, 999)),
                           key_scale=fmt == 1, int2_values=fmt == 2)
        k, v, _ = case.draw(7000 + it, n, 1)
        scale = 2.0 ** gen.integers(-3, 4, size=(n, 1, 1))
        k = synth.to_bf16_representable(k * scale)
        v = synth.to_bf16_representable(v * scale[::-1] + 0.125)
        tok_seq = np.concatenate([np.full(c, b, np.int32) for b, c in enumerate(cnt)])
        tok_pos = np.concatenate([lens0[b] + np.arange(c, dtype=np.int32) for b, c in enumerate(cnt)])
        perm = gen.permutation(n)
        k, v, tok_seq, tok_pos = k[perm], v[perm], tok_seq[perm], tok_pos[perm]
        cache.append(0, _dev(k, torch.bfloat16), _dev(v, torch.bfloat16), _dev(tok_seq), _dev(tok_pos))
        assert case.ctx.novakv_last_device_status() == 0
        assert np.array_equal(cache.seq_lens.cpu().numpy(), np.where(cnt > 0, lens0 + cnt, lens0))
        k64, v64 = k.astype(np.float64), v.astype(np.float64)
        enc = case.oracle.encode(k64, v64) if fmt == 0 else case.oracle.encode_scaled(k64, v64)
        got_k = np.empty_like(enc["kidx"]); got_v = np.empty_like(enc["vidx"])
        for t in range(n):
            kk, vv = cache.load_logical(int(tok_seq[t]), int(tok_pos[t]), 1)
            got_k[t], got_v[t] = kk[0], vv[0]
        check_indices(got_k, enc, "k")
        if fmt < 2:
            check_indices(got_v, enc, "v")
        else:
            codes, meta = case.oracle.encode_values_int2(v64)
            assert np.array_equal(got_v, cache_format.pack_int2(codes))
            got_m = np.stack([cache.load_value_meta(int(tok_seq[t]), int(tok_pos[t]), 1)[0] for t in range(n)])
            assert np.array_equal(got_m, meta)
        if fmt > 0:
            got_s = np.stack([cache.load_scales(int(tok_seq[t]), int(tok_pos[t]), 1)[0] for t in range(n)])
            assert np.array_equal(got_s, enc["kscale"])
