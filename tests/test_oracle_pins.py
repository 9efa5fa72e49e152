"""Pins of the CPU oracle and of the host calibrator against what the paper and the
mathematics fix (no GPU).  Each test names the passage it checks."""
from pathlib import Path

import numpy as np
import pytest

from oracle import novakv_oracle as O
from paper_2608_04074_b200 import cache_format, calib, synth

GOLDEN = Path(__file__).resolve().parent / "golden"


def np_attention(q, k, v, scale):
    """Independent numpy restatement of Eq. "scores" for one query head: q [d], k/v [S][d]."""
    z = (k @ q) * scale
    p = np.exp(z - z.max())
    p /= p.sum()
    return p @ v


def lossless_oracle(laws, n_tok, seed, hkv=1, hg=4, d=64, shift=None):
    """An oracle whose codebooks contain every token's own subvector, so that the quantiser is
    the identity on those tokens; built from float64 (unrounded) transforms."""
    k, v = synth.draw_kv(laws, seed, n_tok)
    q = synth.draw_q(laws, seed + 1, 512)
    kc, vc = synth.draw_kv(laws, seed + 2, 2048)
    if shift is not None:
        k = k + shift
        kc = kc + shift
    g, L = 4, d // 4
    rk = np.empty((hkv, d, d)); rki = np.empty((hkv, d, d)); rv = np.empty((hkv, d, d))
    km = np.empty((hkv, d)); vm = np.empty((hkv, d))
    cbk = np.zeros((hkv, L, 256, g)); cbv = np.zeros((hkv, L, 256, g))
    for h in range(hkv):
        rk[h], rki[h], km[h], _ = calib.key_transform(q[:, h * hg:(h + 1) * hg], kc[:, h])
        o = calib.attention_outputs(q[:, h * hg], kc[:, h], vc[:, h])
        rv[h], _ = calib.value_transform(o)
        vm[h] = vc[:, h].mean(axis=0)
        r = (k[:, h] - km[h]) @ rk[h]
        s = (v[:, h] - vm[h]) @ rv[h]
        # codeword j of every group = token j's subvector; the rest are far away
        cbk[h] += 1e12
        cbv[h] += 1e12
        cbk[h, :, :n_tok, :] = r.reshape(n_tok, L, g).transpose(1, 0, 2)
        cbv[h, :, :n_tok, :] = s.reshape(n_tok, L, g).transpose(1, 0, 2)
    return O.Oracle(rk, rki, rv, km, vm, cbk, cbv), k, v, q


# ---------------------------------------------------------------- transforms (Theorem 1, Prop. 1)

def test_identity_quantiser_reproduces_exact_attention():
    """Sec. 2.2 summary + App. B read path: with a lossless quantiser, encode -> explicit
    dequantise -> inverse transforms -> attention equals plain attention on the raw k, v."""
    laws = synth.draw_layer_laws(synth.LayerShape(4, 1, 64), 5)
    orc, k, v, q = lossless_oracle(laws, 200, 50)
    enc = orc.encode(k, v)
    assert np.array_equal(enc["kidx"][:, 0, :], np.repeat(np.arange(200)[:, None], 16, 1))
    assert np.array_equal(enc["vidx"][:, 0, :], np.repeat(np.arange(200)[:, None], 16, 1))
    k_hat, v_hat = orc.reconstruct(enc["kidx"], enc["vidx"])
    assert np.abs(k_hat - k).max() < 1e-9 * np.abs(k).max()
    assert np.abs(v_hat - v).max() < 1e-11
    qq = q[0]
    out = orc.decode(qq, enc["kidx"], enc["vidx"])
    for h in range(4):
        ref = np_attention(qq[h], k[:, 0], v[:, 0], 1 / 8.0)
        assert np.abs(out[h] - ref).max() < 1e-9


def test_query_fold_products_invariant():
    """App. B "Decoding kernel": (q R_K^{-T}) . ((k - kbar) R_K) = q . (k - kbar)."""
    laws = synth.draw_layer_laws(synth.LayerShape(4, 1, 64), 6)
    k, _ = synth.draw_kv(laws, 60, 300)
    q = synth.draw_q(laws, 61, 300)
    rk, rki, km, lam = calib.key_transform(q, k[:, 0])
    lhs = (q[:, 0] @ rki) @ ((k[:, 0] - km) @ rk).T
    rhs = q[:, 0] @ (k[:, 0] - km).T
    assert np.abs(lhs - rhs).max() < 1e-9 * np.abs(rhs).max()
    # (R_K^{-T})^T R_K = I
    assert np.abs(rki.T @ rk - np.eye(64)).max() < 1e-8


def test_rk_rkT_equals_mq_and_coefficients_decorrelated():
    """Theorem 1 text: R_K R_K^T = M_q; the sample second moment of r is Lambda, descending."""
    laws = synth.draw_layer_laws(synth.LayerShape(4, 1, 64), 7)
    k, _ = synth.draw_kv(laws, 70, 1000)
    q = synth.draw_q(laws, 71, 1000)
    rk, rki, km, lam = calib.key_transform(q, k[:, 0])
    mq = q.reshape(-1, 64).T @ q.reshape(-1, 64)
    assert np.abs(rk @ rk.T - mq).max() < 1e-9 * np.abs(mq).max()
    r = (k[:, 0] - km) @ rk
    srr = r.T @ r
    assert np.all(np.diff(lam) <= 1e-9 * lam[0])
    assert np.abs(srr - np.diag(lam)).max() < 1e-8 * lam[0]


def test_mq_identity_reduces_to_pca():
    """Remark after Theorem 1: M_q proportional to I gives mean-centred PCA of the keys."""
    laws = synth.draw_layer_laws(synth.LayerShape(1, 1, 64), 8)
    k, _ = synth.draw_kv(laws, 80, 500)
    q = (3.0 * np.eye(64))[:, None, :]            # Q^T Q = 9 I exactly
    rk, rki, km, lam = calib.key_transform(q, k[:, 0])
    kc = k[:, 0] - k[:, 0].mean(axis=0)
    w, e = np.linalg.eigh(kc.T @ kc)
    e = e[:, ::-1]
    # columns agree up to sign and the factor sqrt(c) = 3
    m = np.abs((rk / 3.0).T @ e)
    assert np.abs(m - np.eye(64)).max() < 1e-6
    assert np.allclose(lam, 9.0 * w[::-1], rtol=1e-9)


def test_generalised_parseval_on_oracle_reconstruction(tiny_case):
    """Prop. 1 with Eq. "qmse" and App. F (GQA): sum_j ||r_j - r^_j||^2 equals
    sum_h ||Q^(h) K^T - Q^(h) K^^T||_F^2 when M_q is built from those queries."""
    c = tiny_case
    wl, laws, cal, orc = c["wl"], c["laws"], c["cal"], c["oracle"]
    q_cal = synth.draw_q(laws, 1000 * wl.seed + 3, wl.calib_tokens)     # the calibration queries
    k, v = c["k"][:256].astype(np.float64), c["v"][:256].astype(np.float64)
    enc = orc.encode(k, v)
    r = orc.coefficients(k, "k")[:, 0]
    r_hat = orc.cb_k[0][np.arange(16)[None, :], enc["kidx"][:, 0, :]].reshape(256, 64)
    k_hat, _ = orc.reconstruct(enc["kidx"], enc["vidx"])
    lhs = np.sum((r - r_hat) ** 2)
    qq = q_cal.reshape(-1, 64)
    rhs = np.sum((qq @ (k[:, 0] - k_hat[:, 0]).T) ** 2)
    assert abs(lhs - rhs) < 2e-4 * rhs          # tables are float32 at the boundary
    # and it is a real quantiser: the error is not zero
    assert lhs > 0


def test_transposed_synthesis_would_fail_parseval(tiny_case):
    """Guard: Parseval distinguishes R_K^{-T} from its transpose (a transposed operand fails)."""
    c = tiny_case
    orc = c["oracle"]
    bad = O.Oracle(orc.rk, orc.rk_inv_t.transpose(0, 2, 1).copy(), orc.rv, orc.k_mean, orc.v_mean,
                   orc.cb_k, orc.cb_v)
    k, v = c["k"][:64].astype(np.float64), c["v"][:64].astype(np.float64)
    enc = orc.encode(k, v)
    good_k, _ = orc.reconstruct(enc["kidx"], enc["vidx"])
    bad_k, _ = bad.reconstruct(enc["kidx"], enc["vidx"])
    assert np.abs(good_k - bad_k).max() > 1e-3 * np.abs(good_k).max()


# ---------------------------------------------------------------- values (Corollary 1)

def test_value_transform_orthogonal_and_mo_identity():
    """Corollary 1 + "Second moment of the attention outputs": R_V^T R_V = I and
    V^T (S^T S) V = sum_i o_i^T o_i."""
    laws = synth.draw_layer_laws(synth.LayerShape(4, 1, 64), 9)
    k, v = synth.draw_kv(laws, 90, 150)
    q = synth.draw_q(laws, 91, 40)[:, 0]
    z = q @ k[:, 0].T / 8.0
    s = np.exp(z - z.max(axis=1, keepdims=True))
    s /= s.sum(axis=1, keepdims=True)
    o = calib.attention_outputs(q, k[:, 0], v[:, 0])
    mo_def = v[:, 0].T @ (s.T @ s) @ v[:, 0]
    assert np.abs(o.T @ o - mo_def).max() < 1e-10 * np.abs(mo_def).max()
    rv, lam = calib.value_transform(o)
    assert np.abs(rv.T @ rv - np.eye(64)).max() < 1e-12
    assert np.all(np.diff(lam) <= 1e-12)


def test_value_offset_is_exact(tiny_case):
    """Remark after Corollary 1: a shared value offset is added back to the output exactly."""
    c = tiny_case
    orc = c["oracle"]
    enc = orc.encode(c["k"][:128].astype(np.float64), c["v"][:128].astype(np.float64))
    o0 = orc.decode(c["q"], enc["kidx"], enc["vidx"])
    shift = np.linspace(-1, 1, 64)[None, :]
    orc2 = O.Oracle(orc.rk, orc.rk_inv_t, orc.rv, orc.k_mean, orc.v_mean + shift, orc.cb_k, orc.cb_v)
    o1 = orc2.decode(c["q"], enc["kidx"], enc["vidx"])
    assert np.abs(o1 - (o0 + shift)).max() < 1e-12


# ---------------------------------------------------------------- grouping (Theorem 2)

def test_grouping_toy_example_from_figure():
    """Fig. "groupings" (c): d=12, g=4, L=3, coordinate i (by decreasing variance) -> group i mod L."""
    gold = np.loadtxt(GOLDEN / "grouping_toy.txt", dtype=int)
    var = np.arange(12, 0, -1).astype(float)         # already sorted by decreasing variance
    order = calib.equalizing_order(var, 3)
    group_of_coord = np.empty(12, int)
    for pos, coord in enumerate(order):
        group_of_coord[coord] = pos // 4
    assert np.array_equal(group_of_coord, gold)
    assert list(order) == [0, 3, 6, 9, 1, 4, 7, 10, 2, 5, 8, 11]
    # an unsorted spectrum is ranked first (stable on ties)
    var2 = np.array([1.0, 8.0, 8.0, 3.0])
    assert list(calib.equalizing_order(var2, 2)) == [1, 3, 2, 0]


def test_volume_identities_and_spread_ordering():
    """Sec. 4: prod_l v_l = prod_i sigma_i^2 for every partition; AM-GM on v_l^(1/g); on the
    i^-1.5 spectrum spread(equalizing) < spread(random) < spread(sorted) (App. D)."""
    d, g, L = 128, 4, 32
    var = np.arange(1, d + 1, dtype=float) ** -1.5
    logv = np.log(var)
    gen = np.random.default_rng(0)
    parts = {
        "equalizing": calib.equalizing_order(var, L).reshape(L, g),
        "sorted": np.arange(d).reshape(L, g),
        "random": gen.permutation(d).reshape(L, g),
    }
    spread = {}
    for name, p in parts.items():
        lv = logv[p].sum(axis=1)
        assert abs(lv.sum() - logv.sum()) < 1e-9
        am = np.exp(lv / g).sum()
        gm = L * np.exp(logv.sum() / d)
        assert am >= gm * (1 - 1e-12)
        spread[name] = lv.max() - lv.min()
    assert spread["equalizing"] < spread["random"] < spread["sorted"]


# ---------------------------------------------------------------- rate (Sec. 5 "Bit rate")

def test_rate_and_store_arithmetic():
    gold = {}
    for line in (GOLDEN / "paper_arithmetic.txt").read_text().splitlines():
        line = line.split("#")[0].split()
        if len(line) == 2:
            gold[line[0]] = float(line[1])
    assert cache_format.bits_per_element(128) == (2.0, 2.0)
    assert cache_format.bits_per_element(64) == (2.0, 2.0)
    bk, bv = cache_format.bits_per_element(128, key_scale_bits=16, value_meta_bits=32)
    assert bk == gold["bpe_keys_deployed"] and bv == gold["bpe_values_deployed"]
    assert (bk + bv) / 2 == gold["bpe_mean_deployed"]
    assert cache_format.table_scalars(128) == gold["store_scalars_d128"]
    assert 3 * 128 * 128 == gold["store_transforms_d128"]
    assert 32 * 256 * 4 == gold["store_codebooks_d128"]
    assert cache_format.table_scalars(128, True) == gold["store_scalars_d128"] + 32768
    assert 2 * 128 * 2 == gold["bf16_bytes_per_token_per_kv_head"]
    assert cache_format.index_bytes_per_token_per_kv_head(128) == 64
    assert cache_format.index_bytes_per_token_per_kv_head(64) == 32


# ---------------------------------------------------------------- codebooks (Algorithm 3)

def test_lloyd_monotone_and_centroid_is_cell_mean(tiny_case):
    dist = tiny_case["cal"].info["key_distortion"][0]        # [L][iters]
    assert np.all(np.diff(dist, axis=1) <= 1e-9 * dist[:, :1])
    gen = np.random.default_rng(3)
    x = gen.standard_normal((1, 3000, 4)) * np.array([2.0, 1.0, 0.5, 0.25])
    init = x[0, :256].copy()[None]
    c1, _ = calib._lloyd_c(x, init, 1)
    d2 = ((x[0][:, None, :] - init[0][None, :, :]) ** 2).sum(-1)
    a = d2.argmin(axis=1)
    for c in range(256):
        assert np.allclose(c1[0, c], x[0][a == c].mean(axis=0), atol=1e-12)


def test_shannon_lower_bound_on_fresh_gaussians():
    """App. G "Low-rate version": E||r_G - Q(r_G)||^2 >= g v^(1/g) 2^(-2b) for independent
    Gaussians, any quantiser with g*b bits (here g=4, b=2)."""
    gen = np.random.default_rng(4)
    sig2 = np.array([1.0, 0.6, 0.4, 0.3])
    x = gen.standard_normal((1, 20000, 4)) * np.sqrt(sig2)
    cb, _ = calib._lloyd_c(x, x[:, :256].copy(), 15)
    fresh = gen.standard_normal((20000, 4)) * np.sqrt(sig2)
    d2 = ((fresh[:, None, :] - cb[0][None, :, :]) ** 2).sum(-1).min(axis=1)
    bound = 4 * np.prod(sig2) ** 0.25 * 2.0 ** (-4)
    assert d2.mean() >= bound * 0.97
    assert d2.mean() < 4 * bound           # and the codebook is not useless


# ---------------------------------------------------------------- encode (Sec. 2.2, App. B)

def test_search_matches_independent_brute_force(tiny_case):
    c = tiny_case
    orc = c["oracle"]
    coef = orc.coefficients(c["k"][:300].astype(np.float64), "k")[:, 0]
    idx, gap = orc.search(coef, 0, "k")
    cb = orc.cb_k[0]                                         # [L][C][g]
    x = coef.reshape(300, 16, 1, 4)
    d2 = ((x - cb[None]) ** 2).sum(-1)                       # [n][L][C] float64
    ref = d2.argmin(axis=2)
    assert np.array_equal(idx, ref)
    srt = np.sort(d2, axis=2)
    assert np.allclose(gap, (srt[:, :, 1] - srt[:, :, 0]) / srt[:, :, 0], rtol=1e-9)


def test_search_tie_break_and_exact_hits():
    d, g, L, C = 8, 4, 2, 256
    gen = np.random.default_rng(5)
    cb = gen.standard_normal((1, L, C, g)).astype(np.float32).astype(np.float64)
    cb[0, 0, 200] = cb[0, 0, 17]            # duplicate codeword: the lower index must win
    cb[0, 1, 5] = cb[0, 1, 250]
    eye = np.eye(d)[None]
    orc = O.Oracle(eye, eye, eye, np.zeros((1, d)), np.zeros((1, d)), cb, cb)
    coef = np.concatenate([cb[0, 0, 200], cb[0, 1, 250]])[None, :]
    idx, gap = orc.search(coef, 0, "k")
    assert idx.tolist() == [[17, 5]]
    assert gap.tolist() == [[0.0, 0.0]]
    # equidistant between two codewords: first minimum wins
    cb2 = np.full((1, L, C, g), 100.0)
    cb2[0, :, 3] = [1, 0, 0, 0]
    cb2[0, :, 9] = [-1, 0, 0, 0]
    orc2 = O.Oracle(eye, eye, eye, np.zeros((1, d)), np.zeros((1, d)), cb2, cb2)
    idx, gap = orc2.search(np.zeros((1, d)), 0, "v")
    assert idx.tolist() == [[3, 3]] and gap.tolist() == [[0.0, 0.0]]
    # every codeword encodes to itself
    x = np.concatenate([cb[0, 0], cb[0, 1]], axis=1)          # [C][d]
    idx, _ = orc.search(x, 0, "k")
    want = np.arange(C)
    want0 = want.copy(); want0[200] = 17
    want1 = want.copy(); want1[250] = 5
    assert np.array_equal(idx[:, 0], want0) and np.array_equal(idx[:, 1], want1)


def test_encode_equals_coefficients_then_search(tiny_case):
    c = tiny_case
    orc = c["oracle"]
    k, v = c["k"][:100].astype(np.float64), c["v"][:100].astype(np.float64)
    enc = orc.encode(k, v)
    # coefficients pinned to numpy
    r = (k[:, 0] - orc.k_mean[0]) @ orc.rk[0]
    s = (v[:, 0] - orc.v_mean[0]) @ orc.rv[0]
    assert np.allclose(orc.coefficients(k, "k")[:, 0], r, rtol=1e-12, atol=1e-9)
    ik, _ = orc.search(orc.coefficients(k, "k")[:, 0], 0, "k")
    iv, _ = orc.search(orc.coefficients(v, "v")[:, 0], 0, "v")
    assert np.array_equal(enc["kidx"][:, 0], ik) and np.array_equal(enc["vidx"][:, 0], iv)
    d2 = ((s.reshape(100, 16, 1, 4) - orc.cb_v[0][None]) ** 2).sum(-1)
    assert np.array_equal(enc["vidx"][:, 0], d2.argmin(axis=2))
    d2k = ((r.reshape(100, 16, 1, 4) - orc.cb_k[0][None]) ** 2).sum(-1)
    assert np.array_equal(enc["kidx"][:, 0], d2k.argmin(axis=2))


# ---------------------------------------------------------------- decode (Eq. "scores", Lemma S1)

def test_decode_equals_numpy_on_explicit_dequantisation(tiny_case):
    c = tiny_case
    orc = c["oracle"]
    enc = orc.encode(c["k"].astype(np.float64), c["v"].astype(np.float64), with_gaps=False)
    out = orc.decode(c["q"], enc["kidx"], enc["vidx"])
    ar = np.arange(16)[None, :]
    r_hat = orc.cb_k[0][ar, enc["kidx"][:, 0, :]].reshape(-1, 64)
    s_hat = orc.cb_v[0][ar, enc["vidx"][:, 0, :]].reshape(-1, 64)
    k_hat = r_hat @ orc.rk_inv_t[0].T + orc.k_mean[0]
    v_hat = s_hat @ orc.rv[0].T + orc.v_mean[0]
    for h in range(4):
        ref = np_attention(c["q"][h].astype(np.float64), k_hat, v_hat, 1 / 8.0)
        assert np.abs(out[h] - ref).max() < 1e-12
    # the GPU path's algebra (folded query, dropped mean, transform-domain accumulation) must agree
    for h in range(4):
        qf = c["q"][h].astype(np.float64) @ orc.rk_inv_t[0]
        z = (r_hat @ qf) / 8.0
        p = np.exp(z - z.max()); p /= p.sum()
        alt = (p @ s_hat) @ orc.rv[0].T + orc.v_mean[0]
        assert np.abs(out[h] - alt).max() < 1e-10


def test_lemma_s1_key_offset_invariance(tiny_case):
    """Lemma S1: a constant added to every key leaves the attention output unchanged."""
    c = tiny_case
    orc = c["oracle"]
    enc = orc.encode(c["k"][:300].astype(np.float64), c["v"][:300].astype(np.float64), with_gaps=False)
    o0 = orc.decode(c["q"], enc["kidx"], enc["vidx"])
    shift = np.linspace(-3, 5, 64)[None, :]
    orc2 = O.Oracle(orc.rk, orc.rk_inv_t, orc.rv, orc.k_mean + shift, orc.v_mean, orc.cb_k, orc.cb_v)
    o1 = orc2.decode(c["q"], enc["kidx"], enc["vidx"])
    assert np.abs(o1 - o0).max() < 1e-11


def test_degenerate_caches(tiny_case):
    c = tiny_case
    orc = c["oracle"]
    enc = orc.encode(c["k"][:50].astype(np.float64), c["v"][:50].astype(np.float64), with_gaps=False)
    _, v_hat = orc.reconstruct(enc["kidx"], enc["vidx"])
    # one-token cache: o = v^_0 exactly
    o = orc.decode(c["q"], enc["kidx"][:1], enc["vidx"][:1])
    assert np.abs(o - v_hat[0, 0][None, :]).max() < 1e-13
    # zero query: all logits equal, o = mean of v^
    o = orc.decode(np.zeros((4, 64)), enc["kidx"], enc["vidx"])
    assert np.abs(o - v_hat[:, 0].mean(axis=0)[None, :]).max() < 1e-13
    # empty cache
    o = orc.decode(c["q"], enc["kidx"][:0], enc["vidx"][:0])
    assert np.all(o == 0)


def test_planted_needle(tiny_case):
    """One key aligned with the query at large gain takes all the attention mass."""
    c = tiny_case
    orc = c["oracle"]
    k = c["k"][:200].astype(np.float64).copy()
    v = c["v"][:200].astype(np.float64)
    enc = orc.encode(k, v, with_gaps=False)
    k_hat, v_hat = orc.reconstruct(enc["kidx"], enc["vidx"])
    needle = 123
    q = np.repeat(((k_hat[needle, 0] - orc.k_mean[0]) * 400.0)[None, :], 4, 0)
    o = orc.decode(q, enc["kidx"], enc["vidx"])
    assert np.abs(o - v_hat[needle, 0][None, :]).max() < 1e-6


def test_gqa_head_mapping():
    """Query head h reads KV head h // (Hq/Hkv) (App. A, GQA)."""
    gen = np.random.default_rng(6)
    k = gen.standard_normal((30, 2, 8)); v = gen.standard_normal((30, 2, 8))
    q = gen.standard_normal((4, 8))
    out = O.attention(q, k, v)
    for h in range(4):
        ref = np_attention(q[h], k[:, h // 2], v[:, h // 2], 1 / np.sqrt(8))
        assert np.abs(out[h] - ref).max() < 1e-13


# ---- key format with a per-token scale (Algorithm 3 "Normalize"; App. B read path; Sec. 5 "Bit rate") ----
def _bf16_values(x):
    """float32 array -> nearest bfloat16 values (ties to even), by integer arithmetic on the bits."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32)


def test_key_scale_is_rms_in_bf16_and_normalised_coefficients_have_unit_rms(tiny_case):
    o = tiny_case["oracle"]
    coef = o.coefficients(tiny_case["k"][:64], "k")[:, 0, :]
    rho, nrm = o.key_scale(coef)
    r32 = coef.astype(np.float32).astype(np.float64)
    rms = np.sqrt((r32 * r32).sum(axis=1) / o.d)            # ||r||_2 / sqrt(d), not / d
    np.testing.assert_array_equal(rho, _bf16_values(rms.astype(np.float32)))
    # quotient in binary32
    np.testing.assert_array_equal(nrm, (coef.astype(np.float32) / rho[:, None]).astype(np.float64))
    # unit RMS up to the bfloat16 rounding of rho (relative 2^-8)
    assert np.abs(np.sqrt((nrm * nrm).mean(axis=1)) - 1.0).max() < 2.0 ** -8 + 1e-6
    # a zero vector keeps scale 1 and zero coefficients
    rho0, nrm0 = o.key_scale(np.zeros((1, o.d)))
    assert rho0[0] == 1.0 and not nrm0.any()


def test_key_scale_power_of_two_equivariance(tiny_case):
    o = tiny_case["oracle"]
    k, v = tiny_case["k"][:48], tiny_case["v"][:48]
    a = o.encode_scaled(k, v, with_gaps=False)
    k4 = o.k_mean[None] + 4.0 * (k - o.k_mean[None])          # exact in binary64
    b = o.encode_scaled(k4, v, with_gaps=False)
    np.testing.assert_array_equal(a["kidx"], b["kidx"])
    np.testing.assert_array_equal(4.0 * a["kscale"], b["kscale"])
    np.testing.assert_array_equal(a["vidx"], b["vidx"])      # values carry no scale


def test_key_scale_one_reduces_to_unscaled_encoder():
    # identity transform, zero mean, keys with entries +-1: r = k, rho = 1 exactly
    d, g, c = 64, 4, 256
    gen = np.random.Generator(np.random.PCG64(5))
    eye = np.eye(d)[None]
    cb = gen.standard_normal((1, d // g, c, g)).astype(np.float32)
    o = O.Oracle(eye, eye, eye, np.zeros((1, d)), np.zeros((1, d)), cb, cb)
    k = gen.choice([-1.0, 1.0], size=(32, 1, d))
    v = gen.standard_normal((32, 1, d))
    a, b = o.encode(k, v, with_gaps=False), o.encode_scaled(k, v, with_gaps=False)
    assert (b["kscale"] == 1.0).all()
    np.testing.assert_array_equal(a["kidx"], b["kidx"])
    np.testing.assert_array_equal(a["vidx"], b["vidx"])


def test_scaled_reconstruction_is_linear_in_rho_and_logits_follow(tiny_case):
    o = tiny_case["oracle"]
    k, v, q = tiny_case["k"][:40], tiny_case["v"][:40], tiny_case["q"]
    e = o.encode_scaled(k, v, with_gaps=False)
    k1, v1 = o.reconstruct(e["kidx"], e["vidx"])              # scale ignored
    ks, vs = o.reconstruct_scaled(e["kidx"], e["vidx"], e["kscale"])
    np.testing.assert_array_equal(v1, vs)
    lin = o.k_mean[None] + e["kscale"][:, :, None].astype(np.float64) * (k1 - o.k_mean[None])
    np.testing.assert_allclose(ks, lin, rtol=0, atol=1e-12 * np.abs(lin).max())
    # read-path identity: q k^ = rho * <q R_K^{-T}, codewords> + q kbar   (one multiply per token)
    qf = q[0] @ o.rk_inv_t[0]
    cw = np.stack([o.cb_k[0, np.arange(o.n_groups), e["kidx"][j, 0]].reshape(-1) for j in range(40)])
    lhs = ks[:, 0, :] @ q[0]
    rhs = e["kscale"][:, 0] * (cw @ qf) + q[0] @ o.k_mean[0]
    np.testing.assert_allclose(lhs, rhs, rtol=0, atol=1e-9 * np.abs(lhs).max())
    # decode on the scaled format = textbook attention on the explicit reconstruction
    out = o.decode_scaled(q, e["kidx"], e["vidx"], e["kscale"])
    hg = q.shape[0] // o.n_kv_heads
    ref = np.stack([np_attention(q[h], ks[:, h // hg, :], vs[:, h // hg, :], 1.0 / np.sqrt(o.d)) for h in range(q.shape[0])])
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-12)


def test_scaled_key_rate_matches_paper_arithmetic():
    gold = {}
    for line in (Path(__file__).parent / "golden" / "paper_arithmetic.txt").read_text().splitlines():
        if line.strip() and not line.startswith("#"):
            name, val = line.split("#")[0].split()
            gold[name] = float(val)
    kb, vb = cache_format.bits_per_element(128, key_scale_bits=16, value_meta_bits=32)
    assert kb == gold["bpe_keys_deployed"] and vb == gold["bpe_values_deployed"]
    assert (kb + vb) / 2 == gold["bpe_mean_deployed"]
    assert cache_format.bits_per_element(128, key_scale_bits=16)[0] - cache_format.bits_per_element(128)[0] == 16 / 128
    # the band's share at 128K context and the total, to the digits the paper prints
    total = cache_format.deployed_bits_per_element(128 * 1024)
    assert round(total - gold["bpe_mean_deployed"], 3) == gold["bpe_band_extra_128k"]
    assert round(total, 2) == gold["bpe_total_deployed_128k"]
    # the band's share vanishes as the context grows and is everything for a context inside the band
    assert cache_format.deployed_bits_per_element(320) == 16.0
    assert cache_format.deployed_bits_per_element(10 ** 9) - gold["bpe_mean_deployed"] < 1e-5


# ---- learned attention sink (App. "Attention sinks in the quantized serving path") ----
def test_sink_closed_forms(tiny_case):
    o = tiny_case["oracle"]
    k, v, q = tiny_case["k"][:50], tiny_case["v"][:50], tiny_case["q"]
    e = o.encode(k, v, with_gaps=False)
    k_hat, v_hat = o.reconstruct(e["kidx"], e["vidx"])
    hq = q.shape[0]
    hg = hq // o.n_kv_heads
    scale = 1.0 / np.sqrt(o.d)
    plain = o.decode(q, e["kidx"], e["vidx"])
    # (a) a sink at -inf is no sink
    np.testing.assert_allclose(o.decode_sink(q, e["kidx"], e["vidx"], np.full(hq, -1e300)), plain, rtol=0, atol=1e-13)
    # (b) the sink only rescales: o_sink = o_plain * L / (L + exp(s)),  L = sum_j exp(z_j)
    sink = np.linspace(-2.0, 3.0, hq)
    got = o.decode_sink(q, e["kidx"], e["vidx"], sink)
    for h in range(hq):
        z = (k_hat[:, h // hg, :] @ q[h]) * scale
        big = np.exp(z).sum()
        np.testing.assert_allclose(got[h], plain[h] * big / (big + np.exp(sink[h])), rtol=0, atol=1e-12)
    # (c) one token: p = 1 / (1 + exp(s - z))
    one = o.decode_sink(q, e["kidx"][:1], e["vidx"][:1], sink)
    for h in range(hq):
        z = (k_hat[0, h // hg, :] @ q[h]) * scale
        np.testing.assert_allclose(one[h], v_hat[0, h // hg, :] / (1.0 + np.exp(sink[h] - z)), rtol=0, atol=1e-12)
    # (d) empty cache: all the mass on the sink
    assert not o.decode_sink(q, e["kidx"][:0], e["vidx"][:0], sink).any()
    # (e) independent numpy restatement on explicit keys/values
    ref = np.empty_like(got)
    for h in range(hq):
        z = np.concatenate([(k_hat[:, h // hg, :] @ q[h]) * scale, [sink[h]]])
        p = np.exp(z - z.max()); p /= p.sum()
        ref[h] = p[:-1] @ v_hat[:, h // hg, :]
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-12)
    np.testing.assert_allclose(O.attention_sink(q, k_hat, v_hat, sink), ref, rtol=0, atol=1e-12)


def test_sink_breaks_key_offset_invariance(tiny_case):
    """With a sink Lemma S1 no longer holds: moving the key mean changes the output unless the sink logit
    moves by q.kbar * scale with it (the correction the read path applies)."""
    o = tiny_case["oracle"]
    k, v, q = tiny_case["k"][:40], tiny_case["v"][:40], tiny_case["q"]
    e = o.encode(k, v, with_gaps=False)
    hq = q.shape[0]
    sink = np.zeros(hq)
    base = o.decode_sink(q, e["kidx"], e["vidx"], sink)
    shift = np.full((1, o.d), 1.0)
    o2 = O.Oracle(o.rk, o.rk_inv_t, o.rv, o.k_mean + shift, o.v_mean, o.cb_k, o.cb_v)
    moved = o2.decode_sink(q, e["kidx"], e["vidx"], sink)
    assert np.abs(moved - base).max() > 1e-3 * np.abs(base).max()
    fixed = o2.decode_sink(q, e["kidx"], e["vidx"], sink + (q @ shift[0]) / np.sqrt(o.d))
    np.testing.assert_allclose(fixed, base, rtol=0, atol=1e-12)


# ---- BF16 sink-plus-recent band (Fig. "Cache layout at decoding position t") ----
def test_banded_decode_limits_and_mixture(tiny_case):
    o = tiny_case["oracle"]
    k, v, q = (np.asarray(tiny_case[n], np.float64) for n in ("k", "v", "q"))
    k, v = k[:200], v[:200]
    e = o.encode(k, v, with_gaps=False)
    hq = q.shape[0]
    hg = hq // o.n_kv_heads
    scale = 1.0 / np.sqrt(o.d)
    # (a) no band: the plain quantised decode
    none = np.zeros(200, bool)
    np.testing.assert_allclose(o.decode_banded(q, e["kidx"], e["vidx"], k, v, none),
                               o.decode(q, e["kidx"], e["vidx"]), rtol=0, atol=1e-13)
    # (b) everything in the band: exact attention on the raw keys and values, the indices are irrelevant
    full = np.ones(200, bool)
    junk = np.zeros_like(e["kidx"])
    exact = np.stack([np_attention(q[h], k[:, h // hg, :], v[:, h // hg, :], scale) for h in range(hq)])
    np.testing.assert_allclose(o.decode_banded(q, junk, junk, k, v, full), exact, rtol=0, atol=1e-12)
    # (c) sink of 64 and 100 recent tokens: an independent mixture of exact and dequantised rows
    mask = np.zeros(200, bool); mask[:64] = True; mask[100:] = True
    k_hat, v_hat = o.reconstruct(e["kidx"], e["vidx"])
    km, vm = np.where(mask[:, None, None], k, k_hat), np.where(mask[:, None, None], v, v_hat)
    ref = np.stack([np_attention(q[h], km[:, h // hg, :], vm[:, h // hg, :], scale) for h in range(hq)])
    got = o.decode_banded(q, e["kidx"], e["vidx"], k, v, mask)
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-12)
    # the band matters: the result moves towards the exact attention
    plain = o.decode(q, e["kidx"], e["vidx"])
    assert np.abs(got - exact).max() < np.abs(plain - exact).max()


# ---- scalar INT2 value codec of the deployed format (Sec. 5 "Bit rate"; App. B read path) ----
def test_int2_value_codec_properties(tiny_case):
    o = tiny_case["oracle"]
    v = np.asarray(tiny_case["v"][:64], np.float64)
    codes, meta = o.encode_values_int2(v)
    assert codes.max() <= 3 and set(np.unique(codes)) == {0, 1, 2, 3}
    scale, zero = meta[..., 0].astype(np.float64), meta[..., 1].astype(np.float64)
    np.testing.assert_array_equal(meta, _bf16_values(meta))                     # both are bfloat16 values
    s = o.coefficients(v, "v").astype(np.float32).astype(np.float64)
    mn, mx = s.min(axis=2), s.max(axis=2)
    np.testing.assert_array_equal(meta[..., 1], _bf16_values(mn.astype(np.float32)))
    # the 4 levels span the token's range: zero ~ min, zero + 3 scale ~ max (bfloat16 slack 2^-8 relative)
    span = mx - mn
    assert (np.abs(zero + 3 * scale - mx) <= 3 * 2.0 ** -8 * (np.abs(scale) * 3 + np.abs(zero)) + 1e-12).all()
    # nearest level: reconstruction error at most half a step, plus the clamp slack at the two ends
    rec = zero[..., None] + scale[..., None] * codes
    err = np.abs(rec - s)
    assert (err <= 0.5 * scale[..., None] * (1 + 1e-6) + 2.0 ** -7 * span[..., None]).all()
    # explicit reconstruction = s^ R_V^T + vbar
    v_hat = o.reconstruct_values_int2(codes, meta)
    np.testing.assert_allclose(v_hat[:, 0, :], rec[:, 0, :] @ o.rv[0].T + o.v_mean[0], rtol=0, atol=1e-12)


def test_int2_value_codec_exact_cases():
    d = 64
    eye = np.eye(d)[None]
    cb = np.zeros((1, d // 4, 256, 4), np.float32)
    o = O.Oracle(eye, eye, eye, np.zeros((1, d)), np.zeros((1, d)), cb, cb)
    gen = np.random.Generator(np.random.PCG64(9))
    want = gen.integers(0, 4, size=(16, 1, d)).astype(np.uint8)
    want[:, 0, 0], want[:, 0, 1] = 0, 3                                      # both ends present
    zero, scale = -1.5, 0.375                                                # bfloat16-representable
    v = zero + scale * want.astype(np.float64)
    codes, meta = o.encode_values_int2(v)
    np.testing.assert_array_equal(codes, want)
    assert (meta[..., 0] == scale).all() and (meta[..., 1] == zero).all()
    np.testing.assert_array_equal(o.reconstruct_values_int2(codes, meta), v)   # exact round trip
    # power-of-two scaling and a bfloat16-exact shift move (scale, zero) and keep the codes
    codes2, meta2 = o.encode_values_int2(4.0 * v + 2.0)
    np.testing.assert_array_equal(codes2, want)
    assert (meta2[..., 0] == 4 * scale).all() and (meta2[..., 1] == 4 * zero + 2.0).all()
    # a constant vector: scale falls back to 1, every code 0, reconstruction = the constant
    c, m = o.encode_values_int2(np.full((1, 1, d), 0.25))
    assert not c.any() and m[0, 0, 0] == 1.0 and m[0, 0, 1] == 0.25
    # ties go to even: a coefficient exactly half way between levels 0 and 1, and between 1 and 2
    vv = zero + scale * want[:1].astype(np.float64)
    vv[0, 0, 2], vv[0, 0, 3] = zero + 0.5 * scale, zero + 1.5 * scale
    ct, _ = o.encode_values_int2(vv)
    assert ct[0, 0, 2] == 0 and ct[0, 0, 3] == 2


def test_int2_equals_product_codebook_with_affine_map(tiny_case):
    """Four 2-bit codes in a byte index the 256-entry product codebook {0,1,2,3}^4: the scalar codec is a
    vector quantiser with that fixed codebook and a per-token affine map (the identity the read path uses)."""
    o = tiny_case["oracle"]
    v = np.asarray(tiny_case["v"][:32], np.float64)
    codes, meta = o.encode_values_int2(v)
    table = np.stack([(np.arange(256) >> (2 * i)) & 3 for i in range(4)], axis=1).astype(np.float64)   # [256][4]
    packed = (codes.reshape(32, o.n_kv_heads, o.d // 4, 4).astype(np.uint32) << (2 * np.arange(4))).sum(axis=3)
    rec_table = table[packed].reshape(32, o.n_kv_heads, o.d)
    np.testing.assert_array_equal(rec_table, codes.astype(np.float64))


def test_deployed_decode_is_textbook_attention(tiny_case):
    o = tiny_case["oracle"]
    k, v, q = (np.asarray(tiny_case[n], np.float64) for n in ("k", "v", "q"))
    k, v = k[:120], v[:120]
    e = o.encode_scaled(k, v, with_gaps=False)
    codes, meta = o.encode_values_int2(v)
    ks, _ = o.reconstruct_scaled(e["kidx"], e["vidx"], e["kscale"])
    vh = o.reconstruct_values_int2(codes, meta)
    hq = q.shape[0]
    hg = hq // o.n_kv_heads
    ref = np.stack([np_attention(q[h], ks[:, h // hg, :], vh[:, h // hg, :], 1.0 / np.sqrt(o.d)) for h in range(hq)])
    np.testing.assert_allclose(o.decode_deployed(q, e["kidx"], e["kscale"], codes, meta), ref, rtol=0, atol=1e-12)
    assert cache_format.bits_per_element(128, key_scale_bits=16, value_meta_bits=32)[1] == 2.25
