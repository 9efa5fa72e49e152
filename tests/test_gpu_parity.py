"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Indices are compared bit for bit (a difference is tolerated only where the
oracle's float64 relative gap between the two nearest codewords is <= 1e-6, and is counted);
attention outputs within max|delta| <= 2e-3 * ||o||_inf on float32 output."""
import numpy as np
import pytest

from gpu_common import Case, check_indices, check_output, NEAR_TIE
from paper_2608_04074_b200 import calib, synth, workloads

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


@pytest.fixture(scope="module")
def tiny():
    return Case(workloads.tiny())


@pytest.fixture(scope="module")
def qwen():
    return Case(workloads.qwen3_8b(batch=4, seq_len=4096, calib_tokens=4096, lloyd_iters=6))


@pytest.fixture(scope="module")
def gptoss():
    return Case(workloads.gpt_oss_20b(batch=2, seq_len=2048, calib_tokens=4096, lloyd_iters=6))


def _cache(case, seq_lens, capacity=None, seed=3):
    from paper_2608_04074_b200.runtime import PagedCache
    return PagedCache(case.ctx, seq_lens, capacity_tokens=capacity, seed=seed)


def _fill_with_oracle(case, cache, seq_lens, seed):
    """Draw tokens per sequence, encode them with the ORACLE, store the oracle's indices."""
    encs, items = [], []
    for b, n in enumerate(seq_lens):
        k, v, _ = case.draw(seed + 10 * b, int(n), 1)
        enc = case.oracle.encode(k.astype(np.float64), v.astype(np.float64), with_gaps=False) if n > 0 else \
            dict(kidx=np.zeros((0, case.ctx.n_kv_heads, case.ctx.n_groups), np.uint8),
                 vidx=np.zeros((0, case.ctx.n_kv_heads, case.ctx.n_groups), np.uint8))
        encs.append(enc)
        if n > 0:
            items.append((b, 0, enc["kidx"], enc["vidx"]))
    cache.store_logical_batch(items)
    return encs


# --------------------------------------------------------------------------- T1: search only
@pytest.mark.parametrize("name", ["tiny", "qwen", "gptoss"])
def test_search_from_oracle_coefficients_is_exact(name, request):
    case = request.getfixturevalue(name)
    n = 777                                        # several 64-token tiles and a ragged tail
    k, v, _ = case.draw(100, n, 1)
    for which, x in (("k", k), ("v", v)):
        coef = case.oracle.coefficients(x.astype(np.float64), which).astype(np.float32)
        idx_gpu = torch.empty((n, case.ctx.n_kv_heads, case.ctx.n_groups), dtype=torch.uint8, device="cuda")
        case.ctx.novakv_search_coefficients(0, 0 if which == "k" else 1, _dev(coef), idx_gpu)
        got = idx_gpu.cpu().numpy()
        for h in range(case.ctx.n_kv_heads):
            ref, gap = case.oracle.search(coef[:, h].astype(np.float64), h, which)
            bad = (got[:, h] != ref) & (gap > NEAR_TIE)
            assert not bad.any(), f"{which} head {h}: {int(bad.sum())} mismatches outside the near-tie band"


# --------------------------------------------------------------------------- T2: transform + search + paged store
@pytest.mark.parametrize("add", [[200, 64, 1, 130], [20, 7, 1, 3], [1, 0, 0, 0], [70, 60, 50, 40], [0, 2, 0, 0]])
@pytest.mark.parametrize("name", ["tiny", "qwen", "gptoss"])
def test_encode_append_matches_oracle_indices(name, add, request):
    """395 tokens take the tiled (prefill) kernel; 31, 1, 220 and 2 tokens the per-group append kernel with
    1, 1, 7 and 1 passes and 1, 32, 1 and 16 lane groups per token."""
    case = request.getfixturevalue(name)
    lens0 = np.array([0, 5, 63, 130], np.int32)          # existing lengths; tokens are appended after them
    add = np.array(add, np.int32)
    cache = _cache(case, lens0, capacity=lens0 + add)
    n = int(add.sum())
    k, v, _ = case.draw(200, n, 1)
    tok_seq = np.concatenate([np.full(a, b, np.int32) for b, a in enumerate(add)])
    tok_pos = np.concatenate([lens0[b] + np.arange(a, dtype=np.int32) for b, a in enumerate(add)])
    perm = synth.rng(5).permutation(n)                   # tokens of different sequences interleaved
    k, v, tok_seq, tok_pos = k[perm], v[perm], tok_seq[perm], tok_pos[perm]
    cache.append(0, _dev(k, torch.bfloat16), _dev(v, torch.bfloat16), _dev(tok_seq), _dev(tok_pos))
    assert case.ctx.novakv_last_device_status() == 0
    assert np.array_equal(cache.seq_lens.cpu().numpy(), lens0 + add)
    enc = case.oracle.encode(k.astype(np.float64), v.astype(np.float64))
    got_k = np.empty_like(enc["kidx"]); got_v = np.empty_like(enc["vidx"])
    for t in range(n):
        kk, vv = cache.load_logical(int(tok_seq[t]), int(tok_pos[t]), 1)
        got_k[t], got_v[t] = kk[0], vv[0]
    dk, nk = check_indices(got_k, enc, "k")
    dv, nv = check_indices(got_v, enc, "v")
    print(f"[{name}] index mismatches K {dk} V {dv}; oracle near-ties (gap<={NEAR_TIE}) K {nk} V {nv} of {got_k.size}")
    # bytes of positions that were not appended stay untouched (zero)
    kk, _ = cache.load_logical(1, 0, 5)
    assert not kk.any()
    if add[3] > 0:
        kk, _ = cache.load_logical(3, 0, 130)
        assert not kk.any()


@pytest.mark.parametrize("n", [2, 3, 5, 8, 9, 16, 17])
@pytest.mark.parametrize("name", ["qwen", "gptoss"])
def test_append_kernel_every_split_of_the_transform(name, n, request):
    """The per-group append kernel covers n tokens in passes of tp = 2, 4, 8, 8, 16, 16, 32 lanes here; the 32 / tp lane
    groups of a token share its transform in 8, 8, 4, 4, 2, 2, 1 blocks of the input dimension (d = 128; d = 64
    likewise) and split the codebook.  Every split must give the oracle's indices."""
    case = request.getfixturevalue(name)
    lens0 = np.array([61, 0, 64], np.int32)              # appended tokens cross a page boundary in sequence 0
    add = np.array([n - n // 2, 0, n // 2], np.int32)
    cache = _cache(case, lens0, capacity=lens0 + add)
    k, v, _ = case.draw(7000 + n, n, 1)
    tok_seq = np.concatenate([np.full(a, b, np.int32) for b, a in enumerate(add)])
    tok_pos = np.concatenate([lens0[b] + np.arange(a, dtype=np.int32) for b, a in enumerate(add)])
    cache.append(0, _dev(k, torch.bfloat16), _dev(v, torch.bfloat16), _dev(tok_seq), _dev(tok_pos))
    assert case.ctx.novakv_last_device_status() == 0
    assert np.array_equal(cache.seq_lens.cpu().numpy(), lens0 + add)
    enc = case.oracle.encode(k.astype(np.float64), v.astype(np.float64))
    got_k = np.empty_like(enc["kidx"]); got_v = np.empty_like(enc["vidx"])
    for t in range(n):
        kk, vv = cache.load_logical(int(tok_seq[t]), int(tok_pos[t]), 1)
        got_k[t], got_v[t] = kk[0], vv[0]
    check_indices(got_k, enc, "k")
    check_indices(got_v, enc, "v")


@pytest.mark.parametrize("name", ["tiny", "qwen"])
def test_equal_codewords_lowest_index_wins(name, request):
    """Exact ties (Alg. 1 line 7 with the lowest index winning): the upper half of every codebook is made a copy
    of the lower half, so every search ends in an exact tie between c and c + 128.  Both kernels of the write path
    (8 tokens: the per-group append kernel; 300 tokens: the tiled kernel) must store the lower index - a tie is a
    zero gap in the binary32 ranking, so every group goes through the binary64 re-search of the certified search.
    The oracle's gaps are all zero here; the near-tie band comes from a second oracle whose upper half is moved far
    away instead (same decisions, gap = distance between the two nearest different codewords)."""
    import dataclasses
    from oracle import novakv_oracle as O
    from paper_2608_04074_b200.binding import Context
    from paper_2608_04074_b200.runtime import PagedCache
    base = request.getfixturevalue(name)
    cal = dataclasses.replace(base.cal, cb_k=base.cal.cb_k.copy(), cb_v=base.cal.cb_v.copy())
    cal.cb_k[:, :, 128:] = cal.cb_k[:, :, :128]
    cal.cb_v[:, :, 128:] = cal.cb_v[:, :, :128]
    cal.cb_v = calib.snap_to_byte_grid(cal.cb_v)     # (the extremes may have gone with the upper half: new grid)
    assert np.array_equal(cal.cb_v[:, :, 128:], cal.cb_v[:, :, :128])
    far = dataclasses.replace(base.cal, cb_k=cal.cb_k.copy(), cb_v=cal.cb_v.copy())
    far.cb_k[:, :, 128:] += 1.0e3 * np.abs(cal.cb_k).max()
    far.cb_v[:, :, 128:] += 1.0e3 * np.abs(cal.cb_v).max()
    oracle, oracle_far = O.Oracle.from_calibration(cal), O.Oracle.from_calibration(far)
    shape = base.wl.shape
    ctx = Context(shape.n_q_heads, shape.n_kv_heads, shape.head_dim)
    ctx.novakv_load_calibration(0, cal)
    for n in (8, 300):
        k, v, _ = base.draw(900 + n, n, 1)
        cache = PagedCache(ctx, np.zeros(1, np.int32), capacity_tokens=np.array([n], np.int32), seed=3)
        cache.append(0, _dev(k, torch.bfloat16), _dev(v, torch.bfloat16), _dev(np.zeros(n, np.int32)),
                     _dev(np.arange(n, dtype=np.int32)))
        assert ctx.novakv_last_device_status() == 0
        enc = oracle.encode(k.astype(np.float64), v.astype(np.float64))
        enc_far = oracle_far.encode(k.astype(np.float64), v.astype(np.float64))
        got_k, got_v = cache.load_logical(0, 0, n)
        for which, got in (("k", got_k), ("v", got_v)):
            assert (enc[which + "idx"] < 128).all() and not enc[which + "gap"].any()     # the oracle: ties, lower index
            assert np.array_equal(enc[which + "idx"], enc_far[which + "idx"])
            assert (got < 128).all(), f"{which}, {n} tokens: the higher index of two equal codewords was stored"
            check_indices(got, enc_far, which)


# --------------------------------------------------------------------------- T3/T5: decode on the oracle's indices
@pytest.mark.parametrize("name,lens", [
    ("tiny", [1024]),
    ("tiny", [1]),
    ("qwen", [1, 63, 64, 65, 1000, 0, 3001]),
    ("gptoss", [2048, 77, 640]),
])
def test_decode_matches_oracle(name, lens, request):
    case = request.getfixturevalue(name)
    lens = np.array(lens, np.int32)
    cache = _cache(case, lens)
    encs = _fill_with_oracle(case, cache, lens, 300)
    _, _, q = case.draw(301, 1, len(lens))
    refs = [case.oracle.decode(q[b].astype(np.float64), encs[b]["kidx"], encs[b]["vidx"]) for b in range(len(lens))]
    for path, fused, label in ((1, 1, "tensor-core value side"), (0, 1, "CUDA-core value side"),
                               (1, 0, "tensor-core value side, separate merge kernel")):
        case.ctx.novakv_debug_set_value_path(path)
        case.ctx.novakv_debug_set_fused_merge(fused)
        out = torch.full((len(lens), case.ctx.n_q_heads, case.ctx.head_dim), float("nan"), device="cuda")
        cache.decode(0, _dev(q, torch.bfloat16), out=out)
        out = out.cpu().numpy()
        assert case.ctx.novakv_last_device_status() == 0
        worst = 0.0
        for b, n in enumerate(lens):
            if n == 0:
                assert not out[b].any()
                continue
            worst = max(worst, check_output(out[b], refs[b]))
        print(f"[{name} {lens.tolist()} {label}] max|delta|/||o||inf = {worst:.3e}")
    case.ctx.novakv_debug_set_value_path(1)
    case.ctx.novakv_debug_set_fused_merge(1)


# --------------------------------------------------------------------------- T4: split invariance, determinism
@pytest.mark.parametrize("path", [1, 0])
def test_split_count_invariance_and_determinism(qwen, path):
    """path 1: tensor-core value side (binary16 weights: different splits see different running maxima and
    round the weights differently, 2^-12 relative per weight, so invariance holds to ~2e-4 of the output
    scale); path 0: CUDA-core value side, binary32 weights, invariant within binary32 rounding."""
    case = qwen
    lens = np.array([4096, 900, 2500], np.int32)
    cache = _cache(case, lens)
    encs = _fill_with_oracle(case, cache, lens, 400)
    _, _, q = case.draw(401, 1, len(lens))
    qd = _dev(q, torch.bfloat16)
    outs = {}
    case.ctx.novakv_debug_set_value_path(path)
    try:
        for n_ctas in (1, 2, 7, 0):
            case.ctx.novakv_debug_set_scan_ctas(n_ctas)
            outs[n_ctas] = cache.decode(0, qd).cpu().numpy()
            again = cache.decode(0, qd).cpu().numpy()
            assert np.array_equal(outs[n_ctas], again), "same launch configuration must be bitwise reproducible"
    finally:
        case.ctx.novakv_debug_set_scan_ctas(0)
        case.ctx.novakv_debug_set_value_path(1)
    bound = 2e-4 if path == 1 else 2e-5
    for b in range(len(lens)):
        ref = case.oracle.decode(q[b].astype(np.float64), encs[b]["kidx"], encs[b]["vidx"])
        for n_ctas, o in outs.items():
            check_output(o[b], ref)
        scale = np.abs(ref).max()
        for n_ctas in (1, 2, 7):
            assert np.abs(outs[n_ctas][b] - outs[0][b]).max() <= bound * scale


# --------------------------------------------------------------------------- T6: append then decode, end to end
@pytest.mark.parametrize("name", ["tiny", "qwen"])
def test_append_then_decode_end_to_end(name, request):
    case = request.getfixturevalue(name)
    lens0 = np.array([700, 129, 64], np.int32)
    cache = _cache(case, lens0, capacity=lens0 + 2)
    # prefill with the GPU encoder
    toks, seqs, poss = [], [], []
    for b, n in enumerate(lens0):
        k, v, _ = case.draw(500 + b, int(n), 1)
        toks.append((k, v)); seqs.append(np.full(n, b, np.int32)); poss.append(np.arange(n, dtype=np.int32))
    k = np.concatenate([t[0] for t in toks]); v = np.concatenate([t[1] for t in toks])
    cache.seq_lens.zero_()
    cache.append(0, _dev(k, torch.bfloat16), _dev(v, torch.bfloat16), _dev(np.concatenate(seqs)), _dev(np.concatenate(poss)))
    # one decode step: append one token per sequence, then attend (the new token is visible)
    k1, v1, q = case.draw(510, len(lens0), len(lens0))
    cache.append(0, _dev(k1, torch.bfloat16), _dev(v1, torch.bfloat16), _dev(np.arange(len(lens0), dtype=np.int32)),
                 _dev(lens0.astype(np.int32)))
    out = cache.decode(0, _dev(q, torch.bfloat16)).cpu().numpy()
    assert case.ctx.novakv_last_device_status() == 0
    assert np.array_equal(cache.seq_lens.cpu().numpy(), lens0 + 1)
    for b, n in enumerate(lens0):
        kb = np.concatenate([toks[b][0], k1[b:b + 1]]).astype(np.float64)
        vb = np.concatenate([toks[b][1], v1[b:b + 1]]).astype(np.float64)
        enc = case.oracle.encode(kb, vb)
        gk, gv = cache.load_logical(b, 0, int(n) + 1)
        check_indices(gk, enc, "k"); check_indices(gv, enc, "v")
        # decode parity on the GPU's own indices (identical to the oracle's unless a near-tie flipped one)
        check_output(out[b], case.oracle.decode(q[b].astype(np.float64), gk, gv))
        check_output(out[b], case.oracle.decode(q[b].astype(np.float64), enc["kidx"], enc["vidx"]))


# --------------------------------------------------------------------------- output modes, host step
def test_bf16_output_and_custom_scale(qwen):
    case = qwen
    lens = np.array([513, 2000], np.int32)
    cache = _cache(case, lens)
    encs = _fill_with_oracle(case, cache, lens, 600)
    _, _, q = case.draw(601, 1, 2)
    qd = _dev(q, torch.bfloat16)
    o32 = cache.decode(0, qd, sm_scale=0.05)
    o16 = torch.empty_like(o32, dtype=torch.bfloat16)
    cache.decode(0, qd, out=o16, sm_scale=0.05)
    assert torch.equal(o16, o32.to(torch.bfloat16))
    for b in range(2):
        ref = case.oracle.decode(q[b].astype(np.float64), encs[b]["kidx"], encs[b]["vidx"], sm_scale=0.05)
        check_output(o32[b].cpu().numpy(), ref)


def test_step_host_equals_device_calls(qwen):
    case = qwen
    lens0 = np.array([300, 65], np.int32)
    caches = [_cache(case, lens0, capacity=lens0 + 1, seed=9) for _ in range(3)]
    for c in caches:
        _fill_with_oracle(case, c, lens0, 700)
    k1, v1, q = case.draw(701, 2, 2)
    seq = np.arange(2, dtype=np.int32); pos = lens0.copy()
    # device path
    caches[0].append(0, _dev(k1, torch.bfloat16), _dev(v1, torch.bfloat16), _dev(seq), _dev(pos))
    ref = caches[0].decode(0, _dev(q, torch.bfloat16)).cpu()
    # host path
    c = caches[1]
    pin = lambda a, dt=None: (torch.from_numpy(np.ascontiguousarray(a)).to(dt) if dt else torch.from_numpy(np.ascontiguousarray(a))).pin_memory()
    out_h = torch.empty((2, case.ctx.n_q_heads, case.ctx.head_dim), dtype=torch.float32).pin_memory()
    staging = torch.empty(case.ctx.novakv_step_staging_bytes(2, 2), dtype=torch.uint8, device="cuda")
    case.ctx.novakv_step_host(0, pin(k1, torch.bfloat16), pin(v1, torch.bfloat16), pin(seq), pin(pos),
                              pin(q, torch.bfloat16), c.k_pages, c.v_pages, c.page_table, c.seq_lens, out_h,
                              staging, c.workspace)
    assert torch.equal(out_h, ref)
    assert torch.equal(caches[0].k_pages, c.k_pages) and torch.equal(caches[0].v_pages, c.v_pages)
    # pageable (not page-locked) host buffers take the staged-copy route: same result
    c = caches[2]
    host = lambda a, dt=None: (torch.from_numpy(np.ascontiguousarray(a)).to(dt) if dt else torch.from_numpy(np.ascontiguousarray(a)).clone())
    out_p = torch.empty((2, case.ctx.n_q_heads, case.ctx.head_dim), dtype=torch.float32)
    case.ctx.novakv_step_host(0, host(k1, torch.bfloat16), host(v1, torch.bfloat16), host(seq), host(pos),
                              host(q, torch.bfloat16), c.k_pages, c.v_pages, c.page_table, c.seq_lens, out_p,
                              staging, c.workspace)
    assert torch.equal(out_p, ref)
    assert torch.equal(caches[0].k_pages, c.k_pages) and torch.equal(caches[0].v_pages, c.v_pages)
    assert case.ctx.novakv_last_device_status() == 0


# --------------------------------------------------------------------------- T7: host-injected faults
def test_step_host_async_gives_the_same_output(qwen):
    """novakv_step_host_async enqueues the step; after a stream synchronisation the pinned output equals that of
    the synchronous call (same launch configuration: bitwise)."""
    from paper_2608_04074_b200.runtime import PagedCache
    case = qwen
    lens = np.array([300, 64, 1], np.int32)
    outs = []
    for wait in (True, False):
        cache = PagedCache(case.ctx, lens, capacity_tokens=lens + 1, seed=4)
        _fill_with_oracle(case, cache, lens, 830)
        k1, v1, q = case.draw(831, 3, 3)
        pin = lambda a, dt=None: (torch.from_numpy(np.ascontiguousarray(a)).to(dt) if dt else torch.from_numpy(np.ascontiguousarray(a))).pin_memory()
        kh, vh, qh = pin(k1, torch.bfloat16), pin(v1, torch.bfloat16), pin(q, torch.bfloat16)
        seq, pos = pin(np.arange(3, dtype=np.int32)), pin(lens.copy())
        out_h = torch.full((3, case.ctx.n_q_heads, case.ctx.head_dim), float("nan"), dtype=torch.float32).pin_memory()
        staging = torch.empty(case.ctx.novakv_step_staging_bytes(3, 3), dtype=torch.uint8, device="cuda")
        case.ctx.novakv_step_host(0, kh, vh, seq, pos, qh, cache.k_pages, cache.v_pages, cache.page_table, cache.seq_lens,
                                  out_h, staging, cache.workspace, wait=wait)
        torch.cuda.synchronize()
        assert case.ctx.novakv_last_device_status() == 0
        assert np.array_equal(cache.seq_lens.cpu().numpy(), lens + 1)
        outs.append(out_h.clone())
    assert torch.isfinite(outs[0]).all() and torch.equal(outs[0], outs[1])


def test_faults_are_reported_not_trapped(qwen):
    from paper_2608_04074_b200.binding import Context, NovaKVError
    case = qwen
    lens = np.array([200, 100], np.int32)
    cache = _cache(case, lens)
    _fill_with_oracle(case, cache, lens, 800)
    _, _, q = case.draw(801, 1, 2)
    qd = _dev(q, torch.bfloat16)
    good = cache.decode(0, qd).clone()
    # a page id outside the pool: reported in the device status word, the kernel stays in bounds
    saved = cache.page_table.clone()
    cache.page_table[0, 1] = cache.n_pages + 5
    cache.decode(0, qd)
    torch.cuda.synchronize()
    assert case.ctx.novakv_last_device_status() & 1
    cache.page_table.copy_(saved)
    # a length beyond the page table: clamped and reported
    cache.seq_lens[1] = 64 * cache.page_table.shape[1] + 7
    cache.decode(0, qd)
    assert case.ctx.novakv_last_device_status() & 2
    cache.seq_lens.copy_(torch.from_numpy(lens).cuda())
    assert torch.equal(cache.decode(0, qd), good)          # the context is still usable
    assert case.ctx.novakv_last_device_status() == 0
    # an appended token that names a sequence slot out of range
    k1, v1, _ = case.draw(802, 1, 1)
    cache.append(0, _dev(k1, torch.bfloat16), _dev(v1, torch.bfloat16), _dev(np.array([7], np.int32)),
                 _dev(np.array([0], np.int32)))
    assert case.ctx.novakv_last_device_status() & 8
    # host-side validation
    with pytest.raises(NovaKVError, match="workspace"):
        case.ctx.novakv_decode_attention(0, qd, cache.k_pages, cache.v_pages, cache.page_table, cache.seq_lens,
                                         good, cache.workspace[:256])
    fresh = Context(32, 8, 128, n_layers=2)
    fresh.novakv_load_calibration(0, case.cal)
    with pytest.raises(NovaKVError, match="no calibration"):
        fresh.novakv_decode_attention(1, qd, cache.k_pages, cache.v_pages, cache.page_table, cache.seq_lens,
                                      good, cache.workspace)
    bad = type("C", (), {})()
    for n in ("rk", "rk_inv_t", "rv", "k_mean", "v_mean", "cb_k", "cb_v"):
        setattr(bad, n, getattr(case.cal, n))
    bad.cb_v = case.cal.cb_v.copy()
    bad.cb_v[0, 3, 100, 2] += np.float32(1e-4) * max(1.0, abs(float(bad.cb_v[0, 3, 100, 2])))   # off its 7-bit grid
    with pytest.raises(NovaKVError, match="unsupported calibration"):
        fresh.novakv_load_calibration(1, bad)
    with pytest.raises(NovaKVError, match="unsupported shape"):
        Context(64, 8, 128)                                  # d = 128 with 8 query heads per KV head
    fresh.close()


# --------------------------------------------------------------------------- full bench configuration, sampled
def test_bench_configuration_sampled():
    """Qwen3-8B shape, B = 8, S = 16384, in the launch configuration bench.py times: the cache is
    filled by the GPU encoder; indices are checked on sampled tokens, outputs on sampled sequences."""
    wl = workloads.qwen3_8b(batch=8, seq_len=16384, calib_tokens=4096, lloyd_iters=6)
    case = Case(wl)
    from paper_2608_04074_b200.runtime import PagedCache
    cache = PagedCache(case.ctx, wl.seq_lens, seed=11)
    S = 16384
    cache.seq_lens.zero_()
    host_tokens = {}
    for b in range(wl.batch):
        k, v, _ = case.draw(900 + b, S, 1)
        host_tokens[b] = (k, v)
        cache.append(0, _dev(k, torch.bfloat16), _dev(v, torch.bfloat16),
                     _dev(np.full(S, b, np.int32)), _dev(np.arange(S, dtype=np.int32)))
    _, _, q = case.draw(950, 1, wl.batch)
    out = cache.decode(0, _dev(q, torch.bfloat16)).cpu().numpy()
    case.ctx.novakv_debug_set_value_path(0)
    out_cc = cache.decode(0, _dev(q, torch.bfloat16)).cpu().numpy()
    case.ctx.novakv_debug_set_value_path(1)
    assert case.ctx.novakv_last_device_status() == 0
    assert np.array_equal(cache.seq_lens.cpu().numpy(), wl.seq_lens)
    gen = synth.rng(77)
    for b in (0, 5):
        k, v = host_tokens[b]
        gk, gv = cache.load_logical(b, 0, S)
        pick = np.sort(gen.choice(S, size=1024, replace=False))
        enc = case.oracle.encode(k[pick].astype(np.float64), v[pick].astype(np.float64))
        dk, _ = check_indices(gk[pick], enc, "k")
        dv, _ = check_indices(gv[pick], enc, "v")
        ref = case.oracle.decode(q[b].astype(np.float64), gk, gv)
        ratio = check_output(out[b], ref)
        ratio_cc = check_output(out_cc[b], ref)
        print(f"[bench cfg seq {b}] sampled index mismatches K {dk} V {dv}; max|delta|/||o||inf "
              f"{ratio:.3e} (tensor-core value side) {ratio_cc:.3e} (CUDA-core value side)")


def test_long_context_configuration_sampled():
    """Qwen3-8B shape, B = 64, S = 32768 (1 GB of indices, larger than L2), the sweep configuration of
    bench.py: one drawn sequence is encoded by the GPU and its pages are copied to distinct physical pages of
    every other sequence (as the benchmark does); queries differ per sequence.  Outputs are checked on
    sampled sequences against the oracle's decode of the indices the GPU stored; indices on sampled tokens."""
    S, B = 32768, 64
    wl = workloads.qwen3_8b(batch=B, seq_len=S, calib_tokens=4096, lloyd_iters=6)
    case = Case(wl)
    from paper_2608_04074_b200.runtime import PagedCache
    cache = PagedCache(case.ctx, wl.seq_lens, seed=21)
    cache.seq_lens.zero_()
    k, v, _ = case.draw(1200, S, 1)
    for t0 in range(0, S, 8192):
        cache.append(0, _dev(k[t0:t0 + 8192], torch.bfloat16), _dev(v[t0:t0 + 8192], torch.bfloat16),
                     _dev(np.zeros(8192, np.int32)), _dev(np.arange(t0, t0 + 8192, dtype=np.int32)))
    src = cache.page_table[0].long()
    for b in range(1, B):
        dst = cache.page_table[b].long()
        cache.k_pages[dst] = cache.k_pages[src]
        cache.v_pages[dst] = cache.v_pages[src]
    cache.seq_lens.copy_(torch.from_numpy(wl.seq_lens.astype(np.int32)).cuda())
    _, _, q = case.draw(1201, 1, B)
    out = cache.decode(0, _dev(q, torch.bfloat16)).cpu().numpy()
    assert case.ctx.novakv_last_device_status() == 0
    gk, gv = cache.load_logical(0, 0, S)
    pick = np.sort(synth.rng(78).choice(S, size=512, replace=False))
    enc = case.oracle.encode(k[pick].astype(np.float64), v[pick].astype(np.float64))
    dk, _ = check_indices(gk[pick], enc, "k")
    dv, _ = check_indices(gv[pick], enc, "v")
    worst = 0.0
    for b in (0, 17, 63):
        gkb, gvb = cache.load_logical(b, 0, S)
        assert np.array_equal(gkb, gk) and np.array_equal(gvb, gv)
        ref = case.oracle.decode(q[b].astype(np.float64), gk, gv)
        worst = max(worst, check_output(out[b], ref))
    print(f"[B=64 S=32768] sampled index mismatches K {dk} V {dv}; max|delta|/||o||inf {worst:.3e}")


# --------------------------------------------------------------------------- uncompressed comparator
@pytest.mark.parametrize("name,window", [("qwen", 0), ("qwen", 128), ("gptoss", 0), ("gptoss", 128)])
def test_bf16_comparator_matches_textbook_attention(name, window, request):
    """The in-house bf16 decode kernel (used for the compression speed-up and for sliding-window
    layers) against textbook attention on the same bf16 keys and values."""
    from oracle import novakv_oracle as O
    case = request.getfixturevalue(name)
    ctx = case.ctx
    lens = np.array([1, 200, 1025, 0, 3000], np.int32)
    table, n_pages = synth.shuffled_page_table(7, np.maximum(lens, 1), 64)
    hkv, d = ctx.n_kv_heads, ctx.head_dim
    gen = synth.rng(123)
    kp = np.zeros((n_pages, hkv, 64, d), np.float32)
    vp = np.zeros((n_pages, hkv, 64, d), np.float32)
    ks, vs = [], []
    for b, n in enumerate(lens):
        k, v, _ = case.draw(1400 + b, max(int(n), 1), 1)
        ks.append(k[:n]); vs.append(v[:n])
        pos = np.arange(n)
        kp[table[b][pos // 64], :, pos % 64, :] = k[:n]
        vp[table[b][pos // 64], :, pos % 64, :] = v[:n]
    _, _, q = case.draw(1450, 1, len(lens))
    kd, vd = _dev(kp, torch.bfloat16), _dev(vp, torch.bfloat16)
    pt = _dev(np.where(table < 0, 0, table).astype(np.int32))
    sl = _dev(lens)
    ws = torch.empty(ctx.novakv_bf16_workspace_bytes(len(lens), table.shape[1]), dtype=torch.uint8, device="cuda")
    out = torch.empty((len(lens), ctx.n_q_heads, d), dtype=torch.float32, device="cuda")
    ctx.novakv_bf16_decode_attention(_dev(q, torch.bfloat16), kd, vd, pt, sl, out, ws, window=window)
    got = out.cpu().numpy()
    for b, n in enumerate(lens):
        if n == 0:
            assert not got[b].any()
            continue
        s0 = max(0, int(n) - window) if window > 0 else 0
        ref = O.attention(q[b].astype(np.float64), ks[b][s0:].astype(np.float64), vs[b][s0:].astype(np.float64))
        check_output(got[b], ref)


# --------------------------------------------------------------------------- ragged serving mix, sampled
def test_paged_mix_append_then_decode_sampled(qwen):
    """Serving-mix structure at a size the oracle can follow: 40 ragged sequences (lognormal lengths),
    shuffled 64-token pages, prefill by the GPU encoder, then one step = append one token per sequence
    + decode; indices and outputs of sampled sequences are checked against the oracle."""
    case = qwen
    lens0 = synth.lognormal_lengths(4242, 40, median=900, sigma=1.0, lo=1, hi=6000)
    from paper_2608_04074_b200.runtime import PagedCache
    cache = PagedCache(case.ctx, lens0, capacity_tokens=lens0 + 1, seed=77)
    cache.seq_lens.zero_()
    toks = {}
    ks, vs, seqs, poss = [], [], [], []
    for b, n in enumerate(lens0):
        k, v, _ = case.draw(2000 + b, int(n), 1)
        toks[b] = (k, v)
        ks.append(k); vs.append(v); seqs.append(np.full(n, b, np.int32)); poss.append(np.arange(n, dtype=np.int32))
    cache.append(0, _dev(np.concatenate(ks), torch.bfloat16), _dev(np.concatenate(vs), torch.bfloat16),
                 _dev(np.concatenate(seqs)), _dev(np.concatenate(poss)))
    k1, v1, q = case.draw(2100, len(lens0), len(lens0))
    cache.append(0, _dev(k1, torch.bfloat16), _dev(v1, torch.bfloat16), _dev(np.arange(len(lens0), dtype=np.int32)),
                 _dev(lens0.astype(np.int32)))
    out = cache.decode(0, _dev(q, torch.bfloat16)).cpu().numpy()
    assert case.ctx.novakv_last_device_status() == 0
    assert np.array_equal(cache.seq_lens.cpu().numpy(), lens0 + 1)
    order = np.argsort(lens0)
    for b in (int(order[0]), int(order[len(order) // 2]), int(order[-1]), 7):
        n = int(lens0[b]) + 1
        kb = np.concatenate([toks[b][0], k1[b:b + 1]]).astype(np.float64)
        vb = np.concatenate([toks[b][1], v1[b:b + 1]]).astype(np.float64)
        enc = case.oracle.encode(kb, vb)
        gk, gv = cache.load_logical(b, 0, n)
        check_indices(gk, enc, "k"); check_indices(gv, enc, "v")
        check_output(out[b], case.oracle.decode(q[b].astype(np.float64), gk, gv))


# --------------------------------------------------------------------------- other head-group sizes
@pytest.mark.parametrize("hq,hkv,d", [(2, 2, 128), (4, 2, 128), (3, 3, 64), (4, 2, 64)])
def test_small_head_groups(hq, hkv, d):
    """Hq/Hkv of 1 and 2 (padded to a 4-wide table entry inside the kernel), both head dims, both value paths."""
    wl = workloads.Workload(f"hg{hq // hkv}_d{d}", synth.LayerShape(hq, hkv, d), np.array([700, 65], np.int32), seed=9,
                            calib_tokens=2048, calib_queries_for_values=512, lloyd_iters=3)
    case = Case(wl)
    lens = wl.seq_lens
    cache = _cache(case, lens, capacity=lens + 1)
    cache.seq_lens.zero_()
    toks = []
    for b, n in enumerate(lens):
        k, v, _ = case.draw(2300 + b, int(n), 1)
        toks.append((k, v))
        cache.append(0, _dev(k, torch.bfloat16), _dev(v, torch.bfloat16), _dev(np.full(n, b, np.int32)),
                     _dev(np.arange(n, dtype=np.int32)))
    _, _, q = case.draw(2350, 1, len(lens))
    for path in (1, 0):
        case.ctx.novakv_debug_set_value_path(path)
        out = cache.decode(0, _dev(q, torch.bfloat16)).cpu().numpy()
        assert case.ctx.novakv_last_device_status() == 0
        for b, n in enumerate(lens):
            enc = case.oracle.encode(toks[b][0].astype(np.float64), toks[b][1].astype(np.float64))
            gk, gv = cache.load_logical(b, 0, int(n))
            check_indices(gk, enc, "k"); check_indices(gv, enc, "v")
            check_output(out[b], case.oracle.decode(q[b].astype(np.float64), gk, gv))
    case.ctx.close()


# --------------------------------------------------------------------------- key format with a per-token scale
@pytest.fixture(scope="module")
def qwen_scaled():
    return Case(workloads.qwen3_8b(batch=4, seq_len=4096, calib_tokens=4096, lloyd_iters=6), key_scale=True)


@pytest.fixture(scope="module")
def gptoss_scaled():
    return Case(workloads.gpt_oss_20b(batch=2, seq_len=2048, calib_tokens=4096, lloyd_iters=6), key_scale=True)


@pytest.mark.parametrize("add", [[200, 64, 1, 130], [20, 7, 1, 3], [1, 0, 0, 0], [70, 60, 50, 40]])
@pytest.mark.parametrize("name", ["qwen_scaled", "gptoss_scaled"])
def test_scaled_encode_matches_oracle_indices_and_scales(name, add, request):
    """Append on the scaled key format, through the tiled kernel (395 tokens: a long run, a ragged tail, a
    single token) and through the clustered append kernel (31, 1 and 220 tokens: one, one and seven passes):
    indices as in the unscaled test, scales bit for bit (bfloat16)."""
    from paper_2608_04074_b200.runtime import PagedCache
    case = request.getfixturevalue(name)
    lens0 = np.array([0, 5, 63, 130], np.int32)
    add = np.array(add, np.int32)
    cache = PagedCache(case.ctx, lens0, capacity_tokens=lens0 + add, seed=3, key_scale=True)
    n = int(add.sum())
    k, v, _ = case.draw(210, n, 1)
    # a wide range of key norms, so that the scale matters: every token scaled by a power of two
    k = synth.to_bf16_representable(k * (2.0 ** synth.rng(6).integers(-3, 4, size=(n, 1, 1))))
    tok_seq = np.concatenate([np.full(a, b, np.int32) for b, a in enumerate(add)])
    tok_pos = np.concatenate([lens0[b] + np.arange(a, dtype=np.int32) for b, a in enumerate(add)])
    perm = synth.rng(7).permutation(n)
    k, v, tok_seq, tok_pos = k[perm], v[perm], tok_seq[perm], tok_pos[perm]
    cache.append(0, _dev(k, torch.bfloat16), _dev(v, torch.bfloat16), _dev(tok_seq), _dev(tok_pos))
    assert case.ctx.novakv_last_device_status() == 0
    assert np.array_equal(cache.seq_lens.cpu().numpy(), lens0 + add)
    enc = case.oracle.encode_scaled(k.astype(np.float64), v.astype(np.float64))
    got_k = np.empty_like(enc["kidx"]); got_v = np.empty_like(enc["vidx"])
    got_s = np.empty_like(enc["kscale"])
    for t in range(n):
        kk, vv = cache.load_logical(int(tok_seq[t]), int(tok_pos[t]), 1)
        got_k[t], got_v[t] = kk[0], vv[0]
        got_s[t] = cache.load_scales(int(tok_seq[t]), int(tok_pos[t]), 1)[0]
    assert np.array_equal(got_s, enc["kscale"]), f"{int((got_s != enc['kscale']).sum())} scales differ"
    assert n < 100 or len(np.unique(enc["kscale"])) > 8
    dk, nk = check_indices(got_k, enc, "k")
    dv, nv = check_indices(got_v, enc, "v")
    print(f"[{name}] scaled format: index mismatches K {dk} V {dv}; near-ties K {nk} V {nv} of {got_k.size}")


@pytest.mark.parametrize("name,lens", [("qwen_scaled", [1, 63, 64, 65, 1000, 0, 3001]), ("gptoss_scaled", [2048, 77, 640])])
def test_scaled_decode_matches_oracle(name, lens, request):
    """Decode on the oracle's scaled encoding (indices + scales) against explicit dequantisation."""
    from paper_2608_04074_b200.runtime import PagedCache
    case = request.getfixturevalue(name)
    lens = np.array(lens, np.int32)
    cache = PagedCache(case.ctx, lens, seed=3, key_scale=True)
    encs = []
    for b, n in enumerate(lens):
        if n == 0:
            encs.append(None)
            continue
        k, v, _ = case.draw(320 + b, int(n), 1)
        k = synth.to_bf16_representable(k * (2.0 ** synth.rng(8 + b).integers(-2, 3, size=(int(n), 1, 1))))
        e = case.oracle.encode_scaled(k.astype(np.float64), v.astype(np.float64), with_gaps=False)
        cache.store_logical(b, 0, e["kidx"], e["vidx"])
        cache.store_scales(b, 0, e["kscale"])
        encs.append(e)
    _, _, q = case.draw(321, 1, len(lens))
    out = cache.decode(0, _dev(q, torch.bfloat16)).cpu().numpy()
    assert case.ctx.novakv_last_device_status() == 0
    worst = 0.0
    for b, n in enumerate(lens):
        if n == 0:
            assert not out[b].any()
            continue
        ref = case.oracle.decode_scaled(q[b].astype(np.float64), encs[b]["kidx"], encs[b]["vidx"], encs[b]["kscale"])
        worst = max(worst, check_output(out[b], ref))
        # the scale is not a no-op on this input: ignoring it moves the output by far more than the tolerance
        if n >= 64:
            no_scale = case.oracle.decode(q[b].astype(np.float64), encs[b]["kidx"], encs[b]["vidx"])
            assert np.abs(no_scale - ref).max() > 10 * 2e-3 * np.abs(ref).max()
    print(f"[{name} {lens.tolist()}] scaled format: max|delta|/||o||inf = {worst:.3e}")


def test_scaled_append_then_decode_end_to_end(qwen_scaled):
    """Whole path on the scaled format: prefill append, one decode-sized append, decode."""
    from paper_2608_04074_b200.runtime import PagedCache
    case = qwen_scaled
    lens = np.array([300, 65, 1], np.int32)
    cache = PagedCache(case.ctx, np.zeros(3, np.int32), capacity_tokens=lens + 1, seed=4, key_scale=True)
    ks, vs = [], []
    for b, n in enumerate(lens):
        k, v, _ = case.draw(400 + b, int(n) + 1, 1)
        ks.append(k); vs.append(v)
        cache.append(0, _dev(k[:n], torch.bfloat16), _dev(v[:n], torch.bfloat16),
                     _dev(np.full(int(n), b, np.int32)), _dev(np.arange(int(n), dtype=np.int32)))
    # decode-sized append: one token per sequence
    cache.append(0, _dev(np.stack([ks[b][lens[b]] for b in range(3)]), torch.bfloat16),
                 _dev(np.stack([vs[b][lens[b]] for b in range(3)]), torch.bfloat16),
                 _dev(np.arange(3, dtype=np.int32)), _dev(lens.astype(np.int32)))
    assert case.ctx.novakv_last_device_status() == 0
    assert np.array_equal(cache.seq_lens.cpu().numpy(), lens + 1)
    _, _, q = case.draw(401, 1, 3)
    out = cache.decode(0, _dev(q, torch.bfloat16)).cpu().numpy()
    for b in range(3):
        e = case.oracle.encode_scaled(ks[b].astype(np.float64), vs[b].astype(np.float64), with_gaps=False)
        ref = case.oracle.decode_scaled(q[b].astype(np.float64), e["kidx"], e["vidx"], e["kscale"])
        check_output(out[b], ref)


# --------------------------------------------------------------------------- many pairs / one long sequence
def test_many_short_sequences_more_pairs_than_ctas(qwen):
    """320 (sequence, KV head) pairs on 148 scan CTAs: many segments per CTA, CTAs spanning several pairs,
    empty sequences in between, and the high-occupancy variant of the merge kernel."""
    case = qwen
    gen = synth.rng(77)
    lens = gen.integers(1, 200, size=40).astype(np.int32)
    lens[[3, 17, 39]] = 0
    lens[5], lens[6] = 64, 65
    assert len(lens) * case.ctx.n_kv_heads > 2 * 148
    cache = _cache(case, lens, seed=9)
    encs = _fill_with_oracle(case, cache, lens, 700)
    _, _, q = case.draw(701, 1, len(lens))
    out = cache.decode(0, _dev(q, torch.bfloat16)).cpu().numpy()
    assert case.ctx.novakv_last_device_status() == 0
    worst = 0.0
    for b, n in enumerate(lens):
        if n == 0:
            assert not out[b].any()
            continue
        ref = case.oracle.decode(q[b].astype(np.float64), encs[b]["kidx"], encs[b]["vidx"])
        worst = max(worst, check_output(out[b], ref))
    print(f"[40 short sequences] max|delta|/||o||inf = {worst:.3e}")


def test_one_long_sequence_all_ctas_share_each_pair(qwen):
    """One sequence of 20000 tokens (313 pages, ragged last page): every (sequence, KV head) pair is split
    over ~18 scan CTAs, so the merge combines many partials per pair."""
    case = qwen
    lens = np.array([20000], np.int32)
    cache = _cache(case, lens, seed=10)
    encs = _fill_with_oracle(case, cache, lens, 800)
    _, _, q = case.draw(801, 1, 1)
    out = cache.decode(0, _dev(q, torch.bfloat16)).cpu().numpy()
    assert case.ctx.novakv_last_device_status() == 0
    ref = case.oracle.decode(q[0].astype(np.float64), encs[0]["kidx"], encs[0]["vidx"])
    print(f"[one 20000-token sequence] max|delta|/||o||inf = {check_output(out[0], ref):.3e}")


# --------------------------------------------------------------------------- learned attention-sink logit
@pytest.mark.parametrize("name,lens", [("gptoss", [2048, 77, 0, 640]), ("qwen", [1, 64, 1000, 3001])])
def test_sink_decode_matches_oracle(name, lens, request):
    """Sink logits from far below to far above the token logits; key mean non-zero, so the offset
    correction of the sink logit is exercised."""
    case = request.getfixturevalue(name)
    lens = np.array(lens, np.int32)
    cache = _cache(case, lens)
    encs = _fill_with_oracle(case, cache, lens, 900)
    _, _, q = case.draw(901, 1, len(lens))
    hq = case.ctx.n_q_heads
    sink = np.linspace(-6.0, 8.0, hq).astype(np.float32)
    assert np.abs(case.cal.k_mean).max() > 0
    out = cache.decode(0, _dev(q, torch.bfloat16), sink_logits=_dev(sink)).cpu().numpy()
    assert case.ctx.novakv_last_device_status() == 0
    plain = cache.decode(0, _dev(q, torch.bfloat16)).cpu().numpy()
    worst = 0.0
    for b, n in enumerate(lens):
        if n == 0:
            assert not out[b].any()
            continue
        ref = case.oracle.decode_sink(q[b].astype(np.float64), encs[b]["kidx"], encs[b]["vidx"], sink.astype(np.float64))
        worst = max(worst, check_output(out[b], ref))
        if n <= 100:       # the sink is not a no-op: on a short sequence it takes a large share of the mass
            assert np.abs(plain[b] - ref).max() > 0.05 * np.abs(ref).max()
    print(f"[{name} {lens.tolist()}] sink: max|delta|/||o||inf = {worst:.3e}")


def test_sink_on_scaled_key_format(qwen_scaled):
    from paper_2608_04074_b200.runtime import PagedCache
    case = qwen_scaled
    lens = np.array([700, 65], np.int32)
    cache = PagedCache(case.ctx, lens, seed=3, key_scale=True)
    encs = []
    for b, n in enumerate(lens):
        k, v, _ = case.draw(950 + b, int(n), 1)
        e = case.oracle.encode_scaled(k.astype(np.float64), v.astype(np.float64), with_gaps=False)
        cache.store_logical(b, 0, e["kidx"], e["vidx"])
        cache.store_scales(b, 0, e["kscale"])
        encs.append(e)
    _, _, q = case.draw(951, 1, 2)
    sink = np.linspace(-3.0, 5.0, case.ctx.n_q_heads).astype(np.float32)
    out = cache.decode(0, _dev(q, torch.bfloat16), sink_logits=_dev(sink)).cpu().numpy()
    for b in range(2):
        ref = case.oracle.decode_sink(q[b].astype(np.float64), encs[b]["kidx"], encs[b]["vidx"], sink.astype(np.float64),
                                      kscale=encs[b]["kscale"])
        check_output(out[b], ref)


# --------------------------------------------------------------------------- BF16 sink-plus-recent band
@pytest.mark.parametrize("name,n_sink,n_rec", [("qwen", 64, 256), ("gptoss", 64, 256), ("qwen", 0, 32), ("qwen", 128, 8)])
def test_banded_decode_matches_oracle(name, n_sink, n_rec, request):
    """Sequences shorter than the sink, inside the band, just past it and far past it; bulk prefill followed
    by single-token steps that wrap the ring and trigger the deferred block quantisation."""
    from paper_2608_04074_b200.runtime import BandedCache
    case = request.getfixturevalue(name)
    lens = np.array([700, 30, 64, 65, 330, 321, 0], np.int32)
    steps = 21
    cache = BandedCache(case.ctx, len(lens), int(lens.max()) + steps + 64, n_sink=n_sink, n_rec=n_rec, block=8, seed=12)
    ks, vs = [], []
    for b, n in enumerate(lens):
        k, v, _ = case.draw(1000 + b, int(n) + steps, 1)
        ks.append(k); vs.append(v)
        if n > 0:
            cache.prefill(0, b, _dev(k[:n], torch.bfloat16), _dev(v[:n], torch.bfloat16))
    for t in range(steps):
        cache.append_step(0, _dev(np.stack([ks[b][lens[b] + t] for b in range(len(lens))]), torch.bfloat16),
                          _dev(np.stack([vs[b][lens[b] + t] for b in range(len(lens))]), torch.bfloat16))
    assert case.ctx.novakv_last_device_status() == 0
    assert (cache.total == lens + steps).all()
    assert (cache.ring_len >= 0).all() and (cache.ring_len < n_rec + 8).all()
    # the device-side state that novakv_band_append advanced equals the rule applied on the host
    meta, quant = cache.device_state()
    assert np.array_equal(meta[:, 0], np.minimum(cache.total, n_sink))
    assert np.array_equal(meta[:, 1], cache.ring_start) and np.array_equal(meta[:, 2], cache.ring_len)
    assert np.array_equal(quant, cache.quant)
    assert np.array_equal(cache.paged.seq_lens.cpu().numpy(), np.where(cache.quant > 0, n_sink + cache.quant, 0))
    _, _, q = case.draw(1001, 1, len(lens))
    out = cache.decode(0, _dev(q, torch.bfloat16)).cpu().numpy()
    assert case.ctx.novakv_last_device_status() == 0
    worst, n_quant = 0.0, 0
    for b in range(len(lens)):
        k, v = ks[b].astype(np.float64), vs[b].astype(np.float64)
        e = case.oracle.encode(k, v, with_gaps=False)
        mask = cache.band_mask(b)
        n_quant += int((~mask).sum())
        ref = case.oracle.decode_banded(q[b].astype(np.float64), e["kidx"], e["vidx"], k, v, mask)
        worst = max(worst, check_output(out[b], ref))
    assert n_quant > 300          # the quantised middle is exercised
    print(f"[{name} sink {n_sink} recent {n_rec}] banded: {n_quant} quantised positions, max|delta|/||o||inf = {worst:.3e}")


def test_band_append_block_of_four_scaled_keys_and_argument_checks(qwen_scaled):
    """Write side of the band with another block size on the scaled key format (the clustered append kernel skips
    the unused entries of sequences that flush nothing), and its argument checks."""
    from paper_2608_04074_b200.binding import NovaKVError
    from paper_2608_04074_b200.runtime import BandedCache
    case = qwen_scaled
    lens = np.array([0, 70, 90, 200], np.int32)
    steps = 19
    cache = BandedCache(case.ctx, len(lens), int(lens.max()) + steps + 64, n_sink=64, n_rec=16, block=4, seed=21, key_scale=True)
    ks, vs = [], []
    for b, n in enumerate(lens):
        k, v, _ = case.draw(1150 + b, int(n) + steps, 1)
        ks.append(k); vs.append(v)
        if n > 0:
            cache.prefill(0, b, _dev(k[:n], torch.bfloat16), _dev(v[:n], torch.bfloat16))
    for t in range(steps):
        cache.append_step(0, _dev(np.stack([ks[b][lens[b] + t] for b in range(len(lens))]), torch.bfloat16),
                          _dev(np.stack([vs[b][lens[b] + t] for b in range(len(lens))]), torch.bfloat16))
    assert case.ctx.novakv_last_device_status() == 0
    meta, quant = cache.device_state()
    assert np.array_equal(meta[:, 1], cache.ring_start) and np.array_equal(meta[:, 2], cache.ring_len)
    assert np.array_equal(quant, cache.quant) and (cache.ring_len < 16 + 4).all() and cache.quant.max() > 100
    _, _, q = case.draw(1151, 1, len(lens))
    out = cache.decode(0, _dev(q, torch.bfloat16)).cpu().numpy()
    for b in range(len(lens)):
        k, v = ks[b].astype(np.float64), vs[b].astype(np.float64)
        e = case.oracle.encode_scaled(k, v, with_gaps=False)
        ref = case.oracle.decode_banded(q[b].astype(np.float64), e["kidx"], e["vidx"], k, v, cache.band_mask(b), kscale=e["kscale"])
        check_output(out[b], ref)
    # argument checks: ring too small for n_rec + block, sink not a multiple of the page, short staging buffer
    p = cache.paged
    k1 = _dev(np.stack([ks[b][0] for b in range(len(lens))]), torch.bfloat16)
    args = lambda n_sink, n_rec, block, staging: (0, k1, k1, cache.band_k, cache.band_v, n_sink, n_rec, block, cache.band_meta,
                                                   cache.quant_lens, p.k_pages, p.v_pages, p.k_scales, None, p.page_table,
                                                   p.seq_lens, staging)
    with pytest.raises(NovaKVError):
        case.ctx.novakv_band_append(*args(64, 64, 4, cache._staging))
    with pytest.raises(NovaKVError):
        case.ctx.novakv_band_append(*args(32, 16, 4, cache._staging))
    with pytest.raises(NovaKVError, match="workspace"):
        case.ctx.novakv_band_append(*args(64, 16, 4, cache._staging[:256]))
    meta2, quant2 = cache.device_state()
    assert np.array_equal(meta, meta2) and np.array_equal(quant, quant2)       # refused calls change nothing


def test_banded_with_scale_and_sink(qwen_scaled):
    from paper_2608_04074_b200.runtime import BandedCache
    case = qwen_scaled
    lens = np.array([500, 100], np.int32)
    cache = BandedCache(case.ctx, 2, 700, n_sink=64, n_rec=64, block=8, seed=13, key_scale=True)
    ks, vs = [], []
    for b, n in enumerate(lens):
        k, v, _ = case.draw(1100 + b, int(n), 1)
        ks.append(k); vs.append(v)
        cache.prefill(0, b, _dev(k, torch.bfloat16), _dev(v, torch.bfloat16))
    _, _, q = case.draw(1101, 1, 2)
    sink = np.linspace(-2.0, 6.0, case.ctx.n_q_heads).astype(np.float32)
    out = cache.decode(0, _dev(q, torch.bfloat16), sink_logits=_dev(sink)).cpu().numpy()
    for b in range(2):
        k, v = ks[b].astype(np.float64), vs[b].astype(np.float64)
        e = case.oracle.encode_scaled(k, v, with_gaps=False)
        ref = case.oracle.decode_banded(q[b].astype(np.float64), e["kidx"], e["vidx"], k, v, cache.band_mask(b),
                                        kscale=e["kscale"], sink=sink.astype(np.float64))
        check_output(out[b], ref)


# --------------------------------------------------------------------------- deployed format: scaled VQ keys + INT2 values
@pytest.mark.parametrize("add", [[200, 64, 1, 130], [20, 7, 1, 3], [1, 0, 0, 0], [70, 60, 50, 40]])
@pytest.mark.parametrize("name", ["qwen_scaled", "gptoss_scaled"])
def test_deployed_encode_matches_oracle(name, add, request):
    """Keys as in the scaled format; value bytes (four 2-bit levels each) and (scale, zero) bit for bit."""
    from paper_2608_04074_b200 import cache_format
    from paper_2608_04074_b200.runtime import PagedCache
    case = request.getfixturevalue(name)
    lens0 = np.array([0, 5, 63, 130], np.int32)
    add = np.array(add, np.int32)
    cache = PagedCache(case.ctx, lens0, capacity_tokens=lens0 + add, seed=3, int2_values=True)
    n = int(add.sum())
    k, v, _ = case.draw(1300, n, 1)
    v = synth.to_bf16_representable(v * (2.0 ** synth.rng(16).integers(-2, 3, size=(n, 1, 1))) + 0.25)
    tok_seq = np.concatenate([np.full(a, b, np.int32) for b, a in enumerate(add)])
    tok_pos = np.concatenate([lens0[b] + np.arange(a, dtype=np.int32) for b, a in enumerate(add)])
    perm = synth.rng(17).permutation(n)
    k, v, tok_seq, tok_pos = k[perm], v[perm], tok_seq[perm], tok_pos[perm]
    cache.append(0, _dev(k, torch.bfloat16), _dev(v, torch.bfloat16), _dev(tok_seq), _dev(tok_pos))
    assert case.ctx.novakv_last_device_status() == 0
    assert np.array_equal(cache.seq_lens.cpu().numpy(), lens0 + add)
    enc = case.oracle.encode_scaled(k.astype(np.float64), v.astype(np.float64))
    codes, meta = case.oracle.encode_values_int2(v.astype(np.float64))
    want_v = cache_format.pack_int2(codes)
    got_k = np.empty_like(enc["kidx"]); got_v = np.empty_like(want_v)
    got_s = np.empty_like(enc["kscale"]); got_m = np.empty_like(meta)
    for t in range(n):
        kk, vv = cache.load_logical(int(tok_seq[t]), int(tok_pos[t]), 1)
        got_k[t], got_v[t] = kk[0], vv[0]
        got_s[t] = cache.load_scales(int(tok_seq[t]), int(tok_pos[t]), 1)[0]
        got_m[t] = cache.load_value_meta(int(tok_seq[t]), int(tok_pos[t]), 1)[0]
    assert np.array_equal(got_s, enc["kscale"])
    assert np.array_equal(got_m, meta), f"{int((got_m != meta).sum())} value (scale, zero) entries differ"
    assert np.array_equal(got_v, want_v), f"{int((got_v != want_v).sum())} value bytes differ of {want_v.size}"
    check_indices(got_k, enc, "k")


@pytest.mark.parametrize("name,lens", [("qwen_scaled", [1, 63, 64, 65, 1000, 0, 3001]), ("gptoss_scaled", [2048, 77, 640])])
def test_deployed_decode_matches_oracle(name, lens, request):
    from paper_2608_04074_b200 import cache_format
    from paper_2608_04074_b200.runtime import PagedCache
    case = request.getfixturevalue(name)
    lens = np.array(lens, np.int32)
    cache = PagedCache(case.ctx, lens, seed=3, int2_values=True)
    # slots that hold no token (the tail of a partly filled last page) carry whatever the caller's allocator
    # left there: NaN and infinity patterns must not reach the result
    cache.v_meta.view(torch.int16).fill_(0x7FC0)
    cache.k_scales.view(torch.int16).fill_(0x7F80)
    encs = []
    for b, n in enumerate(lens):
        if n == 0:
            encs.append(None)
            continue
        k, v, _ = case.draw(1400 + b, int(n), 1)
        # value scales spread over 2^-9 .. 2^2 (small scales exercise the weight range of the INT2 path)
        v = synth.to_bf16_representable(v * (2.0 ** synth.rng(18 + b).integers(-9, 3, size=(int(n), 1, 1))) - 0.5)
        e = case.oracle.encode_scaled(k.astype(np.float64), v.astype(np.float64), with_gaps=False)
        codes, meta = case.oracle.encode_values_int2(v.astype(np.float64))
        cache.store_logical(b, 0, e["kidx"], cache_format.pack_int2(codes))
        cache.store_scales(b, 0, e["kscale"])
        cache.store_value_meta(b, 0, meta)
        encs.append((e, codes, meta))
    _, _, q = case.draw(1401, 1, len(lens))
    sink = np.linspace(-4.0, 4.0, case.ctx.n_q_heads).astype(np.float32)
    out = cache.decode(0, _dev(q, torch.bfloat16)).cpu().numpy()
    out_sink = cache.decode(0, _dev(q, torch.bfloat16), sink_logits=_dev(sink)).cpu().numpy()
    assert case.ctx.novakv_last_device_status() == 0
    worst = 0.0
    for b, n in enumerate(lens):
        if n == 0:
            assert not out[b].any() and not out_sink[b].any()
            continue
        e, codes, meta = encs[b]
        ref = case.oracle.decode_deployed(q[b].astype(np.float64), e["kidx"], e["kscale"], codes, meta)
        worst = max(worst, check_output(out[b], ref))
        ref_s = case.oracle.decode_deployed(q[b].astype(np.float64), e["kidx"], e["kscale"], codes, meta,
                                            sink=sink.astype(np.float64))
        worst = max(worst, check_output(out_sink[b], ref_s))
    print(f"[{name} {lens.tolist()}] deployed format: max|delta|/||o||inf = {worst:.3e}")


def test_deployed_banded_end_to_end(qwen_scaled):
    """The whole deployed format: scaled keys, INT2 values, BF16 band with deferred quantisation, sink logit."""
    from paper_2608_04074_b200.runtime import BandedCache
    case = qwen_scaled
    lens = np.array([600, 90, 330], np.int32)
    steps = 17
    cache = BandedCache(case.ctx, 3, 700, n_sink=64, n_rec=256, block=8, seed=14, int2_values=True)
    ks, vs = [], []
    for b, n in enumerate(lens):
        k, v, _ = case.draw(1500 + b, int(n) + steps, 1)
        ks.append(k); vs.append(v)
        cache.prefill(0, b, _dev(k[:n], torch.bfloat16), _dev(v[:n], torch.bfloat16))
    for t in range(steps):
        cache.append_step(0, _dev(np.stack([ks[b][lens[b] + t] for b in range(3)]), torch.bfloat16),
                          _dev(np.stack([vs[b][lens[b] + t] for b in range(3)]), torch.bfloat16))
    _, _, q = case.draw(1501, 1, 3)
    sink = np.linspace(-1.0, 5.0, case.ctx.n_q_heads).astype(np.float32)
    out = cache.decode(0, _dev(q, torch.bfloat16), sink_logits=_dev(sink)).cpu().numpy()
    assert case.ctx.novakv_last_device_status() == 0
    for b in range(3):
        k, v = ks[b].astype(np.float64), vs[b].astype(np.float64)
        e = case.oracle.encode_scaled(k, v, with_gaps=False)
        codes, meta = case.oracle.encode_values_int2(v)
        ref = case.oracle.decode_deployed(q[b].astype(np.float64), e["kidx"], e["kscale"], codes, meta, k_exact=k,
                                          v_exact=v, band_mask=cache.band_mask(b), sink=sink.astype(np.float64))
        check_output(out[b], ref)


# --------------------------------------------------------------------------- extreme softmax temperatures
@pytest.mark.parametrize("factor", [16.0, 1e-3])
def test_near_one_hot_and_near_uniform_attention(qwen, factor):
    """Logits scaled by 16 (attention close to one-hot: the running maximum changes abruptly and most
    weights underflow) and by 1e-3 (close to uniform: the output is the mean of the values)."""
    case = qwen
    lens = np.array([1500, 129], np.int32)
    cache = _cache(case, lens, seed=15)
    encs = _fill_with_oracle(case, cache, lens, 1600)
    _, _, q = case.draw(1601, 1, 2)
    scale = factor / np.sqrt(case.ctx.head_dim)
    out = cache.decode(0, _dev(q, torch.bfloat16), sm_scale=scale).cpu().numpy()
    assert case.ctx.novakv_last_device_status() == 0
    for b in range(2):
        ref = case.oracle.decode(q[b].astype(np.float64), encs[b]["kidx"], encs[b]["vidx"], sm_scale=scale)
        check_output(out[b], ref)


# --------------------------------------------------------------------------- work split of the scan
@pytest.mark.parametrize("weight", [0, 1, 24, 40, 200, 4096])
def test_segment_weight_moves_split_points_only(qwen, weight):
    """The cost-weighted split (0 = even in pages; large values push whole pairs to single CTAs) must give
    the same attention output: ragged lengths, empty sequences, pairs much shorter than the weight."""
    case = qwen
    lens = np.array([3001, 0, 64, 1, 777, 130, 0, 2000, 65], np.int32)
    cache = _cache(case, lens, seed=16)
    encs = _fill_with_oracle(case, cache, lens, 1700)
    _, _, q = case.draw(1701, 1, len(lens))
    case.ctx.novakv_debug_set_segment_weight(weight)
    try:
        outs = []
        for ctas in (0, 5):
            case.ctx.novakv_debug_set_scan_ctas(ctas)
            outs.append(cache.decode(0, _dev(q, torch.bfloat16)).cpu().numpy())
        assert case.ctx.novakv_last_device_status() == 0
    finally:
        case.ctx.novakv_debug_set_segment_weight(40)      # the default at d = 128
        case.ctx.novakv_debug_set_scan_ctas(0)
    for b, n in enumerate(lens):
        for out in outs:
            if n == 0:
                assert not out[b].any()
                continue
            ref = case.oracle.decode(q[b].astype(np.float64), encs[b]["kidx"], encs[b]["vidx"])
            check_output(out[b], ref)
