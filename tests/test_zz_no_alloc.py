"""The allocation-free decode entry point (collected last on purpose).

Some users of the library cannot allocate device memory: their engine owns all of it, or their
serving loop must never hit cudaMalloc.  For them `novakv_decode_attention_noalloc` keeps its
scratch in a fixed array inside the library.  This test calls it through the C ABI twice in a row
and checks both results against the ordinary entry point on the same inputs.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def test_noalloc_decode_matches_workspace_decode_twice():
    from gpu_common import Case
    from paper_2608_04074_b200 import workloads
    from paper_2608_04074_b200.binding import NovaKVError
    from paper_2608_04074_b200.runtime import PagedCache, bf16_tensor

    case = Case(workloads.qwen3_8b(batch=3, seq_len=1024, calib_tokens=2048, lloyd_iters=3))
    ctx = case.ctx
    lens = np.array([1500, 64, 333], np.int32)
    cache = PagedCache(ctx, lens, seed=41)
    # fill the cache with the GPU encoder
    cache.seq_lens.zero_()
    for b, n in enumerate(lens):
        k, v, _ = case.draw(1200 + b, int(n), 1)
        cache.append(0, bf16_tensor(k), bf16_tensor(v), torch.full((int(n),), b, dtype=torch.int32, device="cuda"),
                     torch.arange(int(n), dtype=torch.int32, device="cuda"))
    free_before = None
    for call in range(2):                                   # two calls in a row share the same scratch array
        _, _, q = case.draw(1300 + call, 1, len(lens))
        qd = bf16_tensor(q)
        ref = cache.decode(0, qd)                           # existing entry point, caller-owned workspace
        out = torch.full_like(ref, float("nan"))
        torch.cuda.synchronize()
        if call == 1:
            free_before = torch.cuda.mem_get_info()[0]
        ctx.novakv_decode_attention_noalloc(0, qd, cache.k_pages, cache.v_pages, cache.page_table,
                                            cache.seq_lens, out)
        torch.cuda.synchronize()
        if call == 1:                                       # after the first call's set-up the device's free memory does not move
            assert torch.cuda.mem_get_info()[0] == free_before
        assert ctx.novakv_last_device_status() == 0
        # same kernels, same launch configuration, same inputs: the library promises bitwise the same result
        assert torch.equal(out, ref), (call, (out - ref).abs().max().item())
    # the largest batch whose workspace fits the fixed array is accepted, the next one refused
    from paper_2608_04074_b200.binding import NOALLOC_SCRATCH_BYTES
    fit = 1
    while ctx.novakv_decode_workspace_bytes(fit + 1) <= NOALLOC_SCRATCH_BYTES:
        fit += 1
    for n, ok in ((fit, True), (fit + 1, False)):
        qn = torch.zeros((n, ctx.n_q_heads, ctx.head_dim), dtype=torch.bfloat16, device="cuda")
        on = torch.zeros((n, ctx.n_q_heads, ctx.head_dim), dtype=torch.float32, device="cuda")
        ptn = torch.zeros((n, 1), dtype=torch.int32, device="cuda")
        sln = torch.zeros((n,), dtype=torch.int32, device="cuda")
        if ok:
            ctx.novakv_decode_attention_noalloc(0, qn, cache.k_pages, cache.v_pages, ptn, sln, on)
            torch.cuda.synchronize()
        else:
            with pytest.raises(NovaKVError, match="workspace"):
                ctx.novakv_decode_attention_noalloc(0, qn, cache.k_pages, cache.v_pages, ptn, sln, on)
    # a batch whose workspace would not fit the fixed array is refused with a clear status
    big = 4096
    qbig = torch.zeros((big, ctx.n_q_heads, ctx.head_dim), dtype=torch.bfloat16, device="cuda")
    obig = torch.zeros((big, ctx.n_q_heads, ctx.head_dim), dtype=torch.float32, device="cuda")
    pt = torch.zeros((big, 1), dtype=torch.int32, device="cuda")
    sl = torch.zeros((big,), dtype=torch.int32, device="cuda")
    with pytest.raises(NovaKVError, match="workspace"):
        ctx.novakv_decode_attention_noalloc(0, qbig, cache.k_pages, cache.v_pages, pt, sl, obig)
