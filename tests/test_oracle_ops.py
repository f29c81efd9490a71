"""Pins for the oracle's RMSNorm, RoPE, SiLU gate, argmax, MoE routing and attention."""
import numpy as np
import torch

import npref
from oracle import q4d_oracle as orc
from workload import gen

ONE = 0x3F80


def _bits(v):
    return orc.bf16_round(np.asarray(v, dtype=np.float64))


# ------------------------------------------------------------------ RMSNorm

def test_rmsnorm_unit_weight_gives_unit_rms_and_scale_invariance():
    rng = np.random.default_rng(10)
    x = _bits(rng.standard_normal((4, 256)) * 3.0)
    w1 = np.full(256, ONE, dtype=np.uint16)
    y = orc.bf16_to_f64(orc.rmsnorm(x, w1, 1e-6))
    assert np.allclose(np.sqrt((y * y).mean(-1)), 1.0, atol=4e-3)       # bf16 rounding of 256 terms
    x4 = _bits(orc.bf16_to_f64(x) * 4.0)                                # exact scaling by a power of two
    y4 = orc.rmsnorm(x4, w1, 0.0)
    y0 = orc.rmsnorm(x, w1, 0.0)
    assert np.array_equal(y4, y0)


def test_rmsnorm_matches_numpy_restatement_with_weights_and_eps():
    rng = np.random.default_rng(11)
    x = _bits(rng.standard_normal((3, 128)) * 0.1)
    w = _bits(1.0 + 0.02 * rng.standard_normal(128))
    for eps in (1e-6, 1e-5, 0.5):
        got = orc.rmsnorm(x, w, eps)
        want = npref.bf16_bits(npref.rmsnorm(orc.bf16_to_f64(x), orc.bf16_to_f64(w), eps))
        assert np.array_equal(got, want)
    # eps dominates a zero row: output is exactly zero
    z = np.zeros((1, 128), dtype=np.uint16)
    assert np.all(orc.bf16_to_f64(orc.rmsnorm(z, w, 1e-6)) == 0.0)


# --------------------------------------------------------------------- RoPE

def test_rope_position_zero_is_identity_and_norm_is_preserved():
    tab = gen.rope_table(64, 128, 1e4).numpy()
    rng = np.random.default_rng(12)
    h = _bits(rng.standard_normal(128))
    assert np.array_equal(orc.rope(h, tab[0]), h)
    v = orc.bf16_to_f64(h)
    for pos in (1, 7, 63):
        r = orc.bf16_to_f64(orc.rope(h, tab[pos]))
        assert abs(np.linalg.norm(r) - np.linalg.norm(v)) < 2e-2 * np.linalg.norm(v) / np.sqrt(128) * 4
        # pairwise: each (i, i+64) pair keeps its length up to bf16 rounding
        assert np.allclose(r[:64] ** 2 + r[64:] ** 2, v[:64] ** 2 + v[64:] ** 2, rtol=2e-2, atol=1e-3)


def test_rope_pairs_i_with_i_plus_half_and_turns_the_right_way():
    tab = gen.rope_table(8, 128, 1e4).numpy()
    e = np.zeros(128)
    e[3] = 1.0
    r = orc.bf16_to_f64(orc.rope(_bits(e), tab[5]))
    want = np.zeros(128)
    want[3], want[3 + 64] = tab[5, 3, 0], tab[5, 3, 1]      # (1,0) -> (cos, sin)
    assert np.array_equal(r, npref.rbf(want))
    e2 = np.zeros(128)
    e2[3 + 64] = 1.0
    r2 = orc.bf16_to_f64(orc.rope(_bits(e2), tab[5]))
    want2 = np.zeros(128)
    want2[3], want2[3 + 64] = -tab[5, 3, 1], tab[5, 3, 0]   # (0,1) -> (-sin, cos)
    assert np.array_equal(r2, npref.rbf(want2))


def test_rope_table_angles_and_relative_position_property():
    tab = gen.rope_table(300, 128, 1e6).numpy().astype(np.float64)
    i = np.arange(64)
    assert np.allclose(tab[1, :, 0], np.cos(1e6 ** (-2 * i / 128)), atol=1e-7)
    assert np.allclose(tab[200, :, 1], np.sin(200 * 1e6 ** (-2 * i / 128)), atol=1e-6)
    # <rope(q, m), rope(k, n)> depends only on m - n (checked without bf16 rounding, in fp64)
    rng = np.random.default_rng(13)
    q, k = rng.standard_normal(128), rng.standard_normal(128)

    def rot(v, p):
        c, s = tab[p, :, 0], tab[p, :, 1]
        return np.concatenate([v[:64] * c - v[64:] * s, v[64:] * c + v[:64] * s])

    d1 = rot(q, 17) @ rot(k, 5)
    d2 = rot(q, 212) @ rot(k, 200)
    assert abs(d1 - d2) < 1e-4
    # and the oracle's rotation is that rotation, rounded
    assert np.array_equal(orc.bf16_to_f64(orc.rope(_bits(q), tab[17].astype(np.float32))),
                          npref.rbf(rot(npref.rbf(q), 17)))


# --------------------------------------------------------------------- SiLU

def test_silu_gate_special_values():
    g = np.array([0.0, 30.0, -30.0, 1.0, -1.0, 2.5])
    u = np.ones_like(g)
    h = orc.bf16_to_f64(orc.silu_mul(_bits(g), _bits(u)))
    assert h[0] == 0.0
    assert h[1] == 30.0
    assert abs(h[2]) < 1e-11
    assert h[3] == npref.rbf(np.array([1.0 / (1.0 + np.exp(-1.0))]))[0]
    # silu(x) - silu(-x) = x, up to the two roundings
    assert abs((h[3] - h[4]) - 1.0) < 2 ** -8
    u2 = _bits(np.array([2.0, -3.0, 0.5, 0.0, 4.0, -1.0]))
    h2 = orc.bf16_to_f64(orc.silu_mul(_bits(g), u2))
    assert np.array_equal(h2, npref.rbf(npref.silu(g) * orc.bf16_to_f64(u2)))


# ------------------------------------------------------------------- argmax

def test_argmax_brute_force_and_ties_take_lowest_index():
    rng = np.random.default_rng(14)
    lg = rng.standard_normal((5, 1000)).astype(np.float32)
    lg[1, 17] = lg[1, 900] = 50.0
    lg[2, :] = 0.25
    lg[3, 999] = 60.0
    lg[4, 0] = 60.0
    want = [int(np.argmax(lg[0])), 17, 0, 999, 0]
    assert orc.argmax(lg).tolist() == want


# ---------------------------------------------------------------------- MoE

def test_moe_route_topk_weights_and_ties():
    z = np.zeros(128)
    idx, w = orc.moe_route(z, 8, True)
    assert idx.tolist() == list(range(8)) and np.allclose(w, 1 / 8, atol=1e-15)
    idx, w = orc.moe_route(z, 8, False)
    assert np.allclose(w, 1 / 128, atol=1e-15)
    rng = np.random.default_rng(15)
    z = rng.standard_normal(128)
    z[40] = z[3] = z.max() + 1.0          # tie for the top: lower index first
    idx, w = orc.moe_route(z, 8, True)
    order = sorted(range(128), key=lambda e: (-z[e], e))[:8]
    assert idx.tolist() == order and idx[0] == 3 and idx[1] == 40
    p = npref.softmax(z)[order]
    assert np.allclose(w, p / p.sum(), rtol=1e-13)
    assert np.allclose(w, npref.softmax(z[order]), rtol=1e-13)   # = softmax over the selected logits
    idx2, w2 = orc.moe_route(z, 8, False)
    assert np.allclose(w2, p, rtol=1e-13)


# ---------------------------------------------------------------- attention

def test_attention_head_equals_full_matrix_softmax():
    rng = np.random.default_rng(16)
    for T in (1, 2, 17, 300):
        q = _bits(rng.standard_normal(128))
        K = _bits(rng.standard_normal((T, 128)))
        V = _bits(rng.standard_normal((T, 128)))
        got = orc.attention_head(q, K, V)
        want = npref.bf16_bits(npref.attention(orc.bf16_to_f64(q)[None], orc.bf16_to_f64(K), orc.bf16_to_f64(V))[0])
        assert np.array_equal(got, want), T


def test_attention_degenerate_cases():
    rng = np.random.default_rng(17)
    q = _bits(rng.standard_normal(128))
    v0 = _bits(rng.standard_normal((1, 128)))
    k0 = _bits(rng.standard_normal((1, 128)))
    assert np.array_equal(orc.attention_head(q, k0, v0), v0[0])            # one token -> its value
    K = _bits(rng.standard_normal((40, 128)))
    V = np.repeat(v0, 40, axis=0)
    assert np.array_equal(orc.attention_head(q, K, V), v0[0])              # equal values -> that value
    # a key that dominates the scores wins the softmax
    K2 = K.copy()
    K2[7] = _bits(orc.bf16_to_f64(q) * 50.0)
    V2 = _bits(rng.standard_normal((40, 128)))
    assert np.array_equal(orc.attention_head(q, K2, V2), V2[7])
    # a large common shift of the scores changes nothing (max-subtraction is in place)
    big = _bits(orc.bf16_to_f64(q) * 300.0)
    out = orc.attention_head(big, K, V2)
    assert np.all(np.isfinite(orc.bf16_to_f64(out)))


def test_split_kv_with_log_sum_exp_merge_equals_unsplit():
    rng = np.random.default_rng(18)
    T = 333
    q = npref.rbf(rng.standard_normal(128))
    K = npref.rbf(rng.standard_normal((T, 128)))
    V = npref.rbf(rng.standard_normal((T, 128)))
    parts = []
    for a, b in ((0, 64), (64, 200), (200, 201), (201, 333)):
        s = K[a:b] @ q / np.sqrt(128)
        m = s.max()
        p = np.exp(s - m)
        parts.append((m, p.sum(), p @ V[a:b]))
    M = max(m for m, _, _ in parts)
    num = sum(np.exp(m - M) * acc for m, _, acc in parts)
    den = sum(np.exp(m - M) * l for m, l, _ in parts)
    merged = num / den
    full = npref.softmax(K @ q / np.sqrt(128)) @ V
    assert np.allclose(merged, full, rtol=0, atol=1e-12)
    assert np.array_equal(npref.bf16_bits(merged), orc.attention_head(_bits(q), _bits(K), _bits(V)))


def _paged_setup(rng, lens, nkv, num_blocks, perm=None):
    bs, d = 16, 128
    n = len(lens)
    L = 2
    mb = max((l + 1 + bs - 1) // bs for l in lens)
    ids = list(range(num_blocks)) if perm is None else list(perm)
    bt = np.zeros((n, mb), dtype=np.int32)
    pool = _bits(rng.standard_normal((L, 2, num_blocks, nkv, bs, d)))
    cur = 0
    for r, l in enumerate(lens):
        nb = (l + 1 + bs - 1) // bs
        bt[r, :nb] = ids[cur:cur + nb]
        cur += nb
    return pool, bt


def test_paged_gather_equals_contiguous_layout_under_block_permutation():
    rng = np.random.default_rng(19)
    lens = [0, 15, 16, 37, 100]
    nkv, nb = 2, 24
    pool_a, bt_a = _paged_setup(rng, lens, nkv, nb)
    perm = np.random.default_rng(20).permutation(nb)
    pool_b = np.empty_like(pool_a)
    pool_b[:, :, perm] = pool_a                       # logical block i moves to physical perm[i]
    bt_b = perm[bt_a].astype(np.int32)
    for r, l in enumerate(lens):
        for layer in (0, 1):
            for h in range(nkv):
                ka, va = orc.kv_gather(pool_a, nkv, 16, 128, layer, h, bt_a[r], l + 1)
                kb, vb = orc.kv_gather(pool_b, nkv, 16, 128, layer, h, bt_b[r], l + 1)
                assert np.array_equal(ka, kb) and np.array_equal(va, vb)
                # contiguous layout: token t is row t of the request's blocks laid end to end
                flat = pool_a[layer, 0][bt_a[r], h].reshape(-1, 128)[: l + 1]
                assert np.array_equal(ka, flat)
    q = _bits(rng.standard_normal((len(lens), 4, 128)))
    oa = orc.attention_paged(q, pool_a, 4, nkv, 16, 128, 1, lens, bt_a)
    ob = orc.attention_paged(q, pool_b, 4, nkv, 16, 128, 1, lens, bt_b)
    assert np.array_equal(oa, ob)
    # and equals per-head attention on the gathered contiguous K, V with kv head = q head // G
    for r, l in enumerate(lens):
        for qh in range(4):
            k, v = orc.kv_gather(pool_a, nkv, 16, 128, 1, qh // 2, bt_a[r], l + 1)
            assert np.array_equal(oa[r, qh], orc.attention_head(q[r, qh], k, v))


def test_two_requests_sharing_prefix_blocks_read_the_same_kv():
    rng = np.random.default_rng(21)
    pool, bt = _paged_setup(rng, [40, 40], 2, 8)
    bt[1, :2] = bt[0, :2]                             # first 32 tokens shared
    k0, v0 = orc.kv_gather(pool, 2, 16, 128, 0, 1, bt[0], 32)
    k1, v1 = orc.kv_gather(pool, 2, 16, 128, 0, 1, bt[1], 32)
    assert np.array_equal(k0, k1) and np.array_equal(v0, v1)
