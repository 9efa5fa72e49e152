"""Parity at the sizes the benchmark sweep times (GPU; sampled against the oracle).

The GPT-OSS-shaped layer at B = 16, S = 65536 (d = 64, eight query heads per KV head: the kernel
variant with two head sets) and the paged serving mix (128 ragged sequences, shuffled 64-token
pages, append of one token per sequence then decode) are built exactly as bench.py builds them:
one drawn sequence is encoded by the GPU encoder and its pages are copied to distinct physical
pages of the other sequences; queries differ per sequence.  Indices are compared with the oracle
on sampled tokens, outputs on sampled sequences against the oracle's explicit-dequantisation
decode of the indices the GPU stored.
"""
import numpy as np
import pytest

from gpu_common import Case, check_indices, check_output
from paper_2608_04074_b200 import synth, workloads

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def _fill_shared(case, cache, seq_lens, k, v):
    """Encode (k, v) as the longest sequence and copy its pages to the prefixes of all the others."""
    nmax, b0 = int(max(seq_lens)), int(np.argmax(seq_lens))
    cache.seq_lens.zero_()
    for t0 in range(0, nmax, 8192):
        m = min(8192, nmax - t0)
        cache.append(0, _dev(k[t0:t0 + m], torch.bfloat16), _dev(v[t0:t0 + m], torch.bfloat16),
                     _dev(np.full(m, b0, np.int32)), _dev(np.arange(t0, t0 + m, dtype=np.int32)))
    src = cache.page_table[b0].long()
    for b, n in enumerate(seq_lens):
        if b == b0:
            continue
        npg = (int(n) + 63) // 64
        dst = cache.page_table[b, :npg].long()
        cache.k_pages[dst] = cache.k_pages[src[:npg]]
        cache.v_pages[dst] = cache.v_pages[src[:npg]]
    cache.seq_lens.copy_(torch.from_numpy(np.asarray(seq_lens, np.int32)).cuda())
    return b0


def test_gpt_oss_shape_full_size_sampled():
    """B = 16, S = 65536, Hq = 64, Hkv = 8, d = 64, heavy-tailed key channels (the sweep's GPT-OSS line)."""
    from paper_2608_04074_b200.runtime import PagedCache
    S, B = 65536, 16
    wl = workloads.gpt_oss_20b(batch=B, seq_len=S, calib_tokens=4096, lloyd_iters=6)
    case = Case(wl)
    cache = PagedCache(case.ctx, wl.seq_lens, seed=41)
    k, v, _ = case.draw(3100, S, 1)
    b0 = _fill_shared(case, cache, wl.seq_lens, k, v)
    _, _, q = case.draw(3101, 1, B)
    out = cache.decode(0, _dev(q, torch.bfloat16)).cpu().numpy()
    case.ctx.novakv_debug_set_value_path(0)
    out_cc = cache.decode(0, _dev(q, torch.bfloat16)).cpu().numpy()
    case.ctx.novakv_debug_set_value_path(1)
    assert case.ctx.novakv_last_device_status() == 0
    gk, gv = cache.load_logical(b0, 0, S)
    pick = np.sort(synth.rng(79).choice(S, size=512, replace=False))
    enc = case.oracle.encode(k[pick].astype(np.float64), v[pick].astype(np.float64))
    dk, nk = check_indices(gk[pick], enc, "k")
    dv, nv = check_indices(gv[pick], enc, "v")
    worst = worst_cc = 0.0
    for b in (0, 7, 15):
        gkb, gvb = cache.load_logical(b, 0, S)
        assert np.array_equal(gkb, gk) and np.array_equal(gvb, gv)
        ref = case.oracle.decode(q[b].astype(np.float64), gk, gv)
        worst = max(worst, check_output(out[b], ref))
        worst_cc = max(worst_cc, check_output(out_cc[b], ref))
    print(f"[gpt-oss shape B=16 S=65536] sampled index mismatches K {dk} V {dv} (near-ties K {nk} V {nv}); "
          f"max|delta|/||o||inf {worst:.3e} (tensor-core value side) {worst_cc:.3e} (CUDA-core value side)")
    case.ctx.close()


def test_paged_mix_full_size_sampled():
    """128 sequences, lognormal lengths in [1024, 131072] (median 8192), shuffled 64-token pages, Qwen3-8B KV
    shape: append one new token per sequence, then decode (the sweep's paged serving mix)."""
    from paper_2608_04074_b200.runtime import PagedCache
    wl = workloads.paged_mix(calib_tokens=4096, lloyd_iters=6)
    case = Case(wl)
    lens0 = wl.seq_lens
    n_seq = wl.batch
    cache = PagedCache(case.ctx, lens0, capacity_tokens=lens0 + 64, seed=37)
    nmax = int(lens0.max())
    k, v, _ = case.draw(3200, nmax, 1)
    b0 = _fill_shared(case, cache, lens0, k, v)
    k1, v1, q = case.draw(3201, n_seq, n_seq)
    cache.append(0, _dev(k1, torch.bfloat16), _dev(v1, torch.bfloat16), _dev(np.arange(n_seq, dtype=np.int32)),
                 _dev(lens0.astype(np.int32)))
    out = cache.decode(0, _dev(q, torch.bfloat16)).cpu().numpy()
    assert case.ctx.novakv_last_device_status() == 0
    assert np.array_equal(cache.seq_lens.cpu().numpy(), lens0 + 1)
    # indices: sampled tokens of the drawn sequence, and every appended token
    gk, gv = cache.load_logical(b0, 0, nmax)
    pick = np.sort(synth.rng(80).choice(nmax, size=512, replace=False))
    enc = case.oracle.encode(k[pick].astype(np.float64), v[pick].astype(np.float64))
    dk, _ = check_indices(gk[pick], enc, "k")
    dv, _ = check_indices(gv[pick], enc, "v")
    enc1 = case.oracle.encode(k1.astype(np.float64), v1.astype(np.float64))
    got1k = np.stack([cache.load_logical(b, int(lens0[b]), 1)[0][0] for b in range(n_seq)])
    got1v = np.stack([cache.load_logical(b, int(lens0[b]), 1)[1][0] for b in range(n_seq)])
    check_indices(got1k, enc1, "k"); check_indices(got1v, enc1, "v")
    # outputs: shortest, median, longest and one more sequence
    order = np.argsort(lens0)
    worst = 0.0
    for b in (int(order[0]), int(order[n_seq // 2]), int(order[-1]), 77):
        n = int(lens0[b]) + 1
        gkb, gvb = cache.load_logical(b, 0, n)
        assert np.array_equal(gkb[:n - 1], gk[:n - 1]) and np.array_equal(gkb[n - 1], got1k[b])
        worst = max(worst, check_output(out[b], case.oracle.decode(q[b].astype(np.float64), gkb, gvb)))
    print(f"[paged mix, {n_seq} sequences, lengths {int(lens0.min())}..{nmax}] sampled index mismatches K {dk} V {dv}; "
          f"max|delta|/||o||inf {worst:.3e}")
    case.ctx.close()


def test_dominant_token_with_long_tail():
    """One token far above a long, nearly flat tail (S = 131072): the tail's weights are tiny relative to the
    maximum, yet their mass is not negligible.  Checks that small softmax weights survive the binary16 rounding
    of the tensor-core value side (they are scaled by 2^15 before it)."""
    from paper_2608_04074_b200.runtime import PagedCache
    S = 131072
    wl = workloads.qwen3_8b(batch=1, seq_len=S, calib_tokens=4096, lloyd_iters=6)
    case = Case(wl)
    cache = PagedCache(case.ctx, wl.seq_lens, seed=51)
    k, v, q = case.draw(3300, S, 1)
    # token 12345 of every KV head is made the query direction of that head's first query head, scaled up
    hg = case.ctx.n_q_heads // case.ctx.n_kv_heads
    for h in range(case.ctx.n_kv_heads):
        qq = q[0, h * hg].astype(np.float64)
        k[12345, h] = synth.to_bf16_representable((qq / np.linalg.norm(qq) * 60.0).astype(np.float32))
    _fill_shared(case, cache, wl.seq_lens, k, v)
    gk, gv = cache.load_logical(0, 0, S)
    for sm in (0.02, 1.0 / np.sqrt(128)):
        out = cache.decode(0, _dev(q, torch.bfloat16), sm_scale=sm).cpu().numpy()
        ref = case.oracle.decode(q[0].astype(np.float64), gk, gv, sm_scale=sm)
        r = check_output(out[0], ref)
        print(f"[dominant token, S={S}, sm_scale={sm:.4f}] max|delta|/||o||inf {r:.3e}")
    assert case.ctx.novakv_last_device_status() == 0
    case.ctx.close()
