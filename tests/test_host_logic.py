"""CPU tests of the host logic: the C ABI exports, the cache byte layout, the workloads, and the
N > 1 plumbing under gloo (world size 2)."""
import ctypes
import os
import re
import subprocess
import sys
from pathlib import Path

import numpy as np
import pytest

from paper_2608_04074_b200 import binding, build, cache_format, sharding, synth, workloads

ROOT = Path(__file__).resolve().parent.parent


def test_library_builds_loads_and_exports_every_declared_symbol():
    lib_path = build.build_cuda()
    lib = ctypes.CDLL(str(lib_path))
    header = (ROOT / "include" / "novakv.h").read_text()
    declared = sorted(set(re.findall(r"\b(novakv_[a-z0-9_]+)\s*\(", header)))
    assert "novakv_encode_append" in declared and "novakv_decode_attention" in declared \
        and "novakv_load_calibration" in declared
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in novakv.h but not exported"
    assert sorted(binding.EXPORTED) == declared, "binding.EXPORTED and novakv.h disagree"
    # no compute without a GPU, but the pure host entry points answer
    lib.novakv_status_string.restype = ctypes.c_char_p
    assert lib.novakv_status_string(0) == b"ok"
    assert lib.novakv_status_string(5).startswith(b"workspace")


def test_product_path_never_touches_the_oracle():
    """The package must not import, load or execute anything under oracle/."""
    pkg = ROOT / "paper_2608_04074_b200"
    for f in list(pkg.rglob("*.py")) + list(pkg.rglob("*.cu")) + list(pkg.rglob("*.cuh")) + list(pkg.rglob("*.c")):
        txt = f.read_text()
        assert "novakv_oracle" not in txt and "from oracle" not in txt and "import oracle" not in txt, f


def test_cache_layout_round_trip_and_positions():
    hkv, d = 2, 64
    L = d // 4
    gen = np.random.default_rng(0)
    lens = np.array([130, 5, 64], np.int32)
    table, n_pages = synth.shuffled_page_table(3, lens, 64)
    assert n_pages == 3 + 1 + 1
    used = table[table >= 0]
    assert sorted(used.tolist()) == list(range(n_pages))          # distinct physical pages
    kp, vp = cache_format.alloc_pools(n_pages, hkv, d)
    assert kp.shape[1] * kp.shape[2] == cache_format.page_bytes(hkv, d)
    ref = {}
    for b, n in enumerate(lens):
        k = gen.integers(0, 256, (n, hkv, L), dtype=np.uint8)
        v = gen.integers(0, 256, (n, hkv, L), dtype=np.uint8)
        cache_format.write_tokens(kp, vp, table[b], 0, k, v)
        ref[b] = (k, v)
    for b, n in enumerate(lens):
        k, v = cache_format.read_tokens(kp, vp, table[b], hkv, d, 0, int(n))
        assert np.array_equal(k, ref[b][0]) and np.array_equal(v, ref[b][1])
    # documented byte positions of the chunk layouts (d = 64: L = 16, one 16-byte plane, 2 group blocks)
    b, pos, h, l = 0, 77, 1, 9
    page = table[b][pos // 64]
    t = pos % 64                                       # 13
    j = l ^ (t % 8)                                    # byte of the token's key bytes that holds group l (l < 16)
    k_off = (((t // 32) * 1 + j // 16) * 32 + t % 32) * 16 + j % 16
    assert kp[page, h, k_off] == ref[b][0][pos, h, l]
    fc, bb, fr = (t % 16) % 4, (t % 16) // 4, l % 8
    v_off = (t // 16) * (L * 16) + (fr * 4 + fc) * 8 + ((l // 8) ^ (t % 2)) * 4 + bb   # odd tokens: group blocks swapped
    assert vp[page, h, v_off] == ref[b][1][pos, h, l]
    # every byte of a chunk is hit exactly once
    tt, ll = np.meshgrid(np.arange(64), np.arange(L), indexing="ij")
    for LL in (16, 32):
        tt, ll = np.meshgrid(np.arange(64), np.arange(LL), indexing="ij")
        assert sorted(cache_format.key_offset(tt, ll, LL).ravel().tolist()) == list(range(64 * LL))
        assert sorted(cache_format.value_offset(tt, ll, LL).ravel().tolist()) == list(range(64 * LL))


def test_value_codebook_grid_snap():
    """The declared rounding of value codebooks: every coordinate of a codebook on its own 128-point affine grid
    between its smallest and largest value; idempotent; at most half a step away from the unsnapped value."""
    from paper_2608_04074_b200 import calib
    gen = synth.rng(77)
    cb = (gen.standard_normal((2, 5, 256, 4)) * np.array([0.01, 1.0, 30.0, 1e-6])).astype(np.float32)
    cb[0, 0, :, 2] = 0.25                                   # a constant coordinate stays what it is
    sn = calib.snap_to_byte_grid(cb)
    assert sn.dtype == np.float32 and sn.shape == cb.shape
    assert np.array_equal(calib.snap_to_byte_grid(sn), sn)
    assert np.array_equal(sn[0, 0, :, 2], cb[0, 0, :, 2])
    lo, hi = cb.min(axis=-2, keepdims=True).astype(np.float64), cb.max(axis=-2, keepdims=True).astype(np.float64)
    step = np.where(hi > lo, (hi - lo) / calib.GRID_LEVELS, 1.0)
    assert np.array_equal(sn.min(axis=-2), cb.min(axis=-2)) and np.array_equal(sn.max(axis=-2), cb.max(axis=-2))
    u = (sn.astype(np.float64) - lo) / step
    assert np.abs(u - np.rint(u)).max() < 1e-4 and u.min() >= -1e-4 and u.max() <= calib.GRID_LEVELS + 1e-4
    assert (np.abs(sn.astype(np.float64) - cb) <= 0.5 * step * (1 + 1e-6) + 1e-12).all()
    for h in range(2):
        for l in range(5):
            for i in range(4):
                assert len(np.unique(sn[h, l, :, i])) <= calib.GRID_LEVELS + 1
    # the calibrator applies it to the value codebooks only
    wl = workloads.tiny()
    cal = wl.calibration(wl.laws())
    assert np.array_equal(calib.snap_to_byte_grid(cal.cb_v), cal.cb_v)
    assert not np.array_equal(calib.snap_to_byte_grid(cal.cb_k), cal.cb_k)


def test_workloads_have_the_stated_shapes():
    w = workloads.qwen3_8b()
    assert (w.shape.n_q_heads, w.shape.n_kv_heads, w.shape.head_dim, w.batch) == (32, 8, 128, 8)
    assert w.decode_index_bytes() == 67108864                    # 64 MiB of packed indices at S = 16384
    assert workloads.qwen3_8b(64, 32768).decode_index_bytes() == 1 << 30
    g = workloads.gpt_oss_20b()
    assert (g.shape.n_q_heads, g.shape.n_kv_heads, g.shape.head_dim) == (64, 8, 64)
    assert g.decode_index_bytes() == 268435456
    m = workloads.paged_mix()
    assert m.batch == 128 and m.seq_lens.min() >= 1024 and m.seq_lens.max() <= 131072
    t = workloads.tiny()
    assert (t.shape.hg, t.shape.head_dim, int(t.seq_lens[0])) == (4, 64, 1024)


def test_bf16_rounding_helper_matches_torch():
    torch = pytest.importorskip("torch")
    x = np.random.default_rng(1).standard_normal(10000).astype(np.float32) * 37.0
    ours = synth.to_bf16_representable(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(ours, ref)


def test_shard_sequences_partitions_the_batch():
    for n, w in ((8, 2), (7, 3), (128, 8), (3, 4)):
        parts = [sharding.shard_sequences(n, r, w) for r in range(w)]
        assert np.array_equal(np.concatenate(parts), np.arange(n))
        assert max(len(p) for p in parts) - min(len(p) for p in parts) <= 1


_WORKER = r"""
import os, sys
sys.path.insert(0, sys.argv[1])
import numpy as np, torch, torch.distributed as dist
from paper_2608_04074_b200 import sharding, workloads
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
wl = workloads.paged_mix(n_seq=16)
mine = sharding.shard_sequences(wl.batch, rank, world)
local_bytes = int(wl.seq_lens[mine].astype(np.int64).sum()) * wl.shape.n_kv_heads * 2 * wl.n_groups
total = sharding.sum_over_ranks(local_bytes)
worst = sharding.max_over_ranks(10.0 + rank)
assert total == wl.decode_index_bytes(), (total, wl.decode_index_bytes())
assert worst == 10.0 + world - 1
dist.barrier()
if rank == 0:
    print("OK", world, int(total))
dist.destroy_process_group()
"""


def test_two_rank_gloo_sharding_and_timing_reduction(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29513", OMP_NUM_THREADS="1")
    res = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29513", str(script), str(ROOT)],
                         capture_output=True, text=True, env=env, timeout=300)
    assert res.returncode == 0, res.stdout + res.stderr
    assert "OK 2" in res.stdout


def test_bench_reference_arm_prints_one_json_line():
    import json
    res = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--batch", "2", "--seq-len", "512"],
                         capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stderr
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    r = json.loads(lines[0])
    assert r["impl"] == "reference" and r["value"] > 0 and r["cpu_baseline"]["kind"] == "oracle"
    assert r["e2e"]["h2d_bytes_per_step"] == 0


def test_bench_gpus_flag_launches_ranks():
    """`bench.py --gpus 2` outside a launcher starts two ranks itself (here the CPU reference arm, gloo
    rendezvous on 127.0.0.1) and rank 0 prints one JSON line that says so."""
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                          "--warmup", "0", "--batch", "2", "--seq-len", "512", "--calib-tokens", "1024", "--lloyd-iters", "2"],
                         capture_output=True, text=True, timeout=600, env=env)
    assert res.returncode == 0, res.stdout + res.stderr
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, res.stdout
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["n_gpus"] == 2
    assert out["cpu_baseline"]["cores"] == len(os.sched_getaffinity(0))
