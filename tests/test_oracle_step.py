"""Pins for the oracle's whole decode step: an independent numpy restatement on toy
shapes, batch invariance, physical-layout invariance, and MoE special cases."""
import numpy as np
import pytest
import torch

import npref
from oracle import q4d_oracle as orc
from workload import gen, shapes


def _dense_dict(shape, weights):
    def mat(t):
        return npref.dense_matrix(tuple(orc.to_np(a) for a in t))

    def vec(t):
        return npref.bf16_val(orc.to_np(t))

    out = {"layers": [], "final_norm": vec(weights["final_norm"]), "embed": mat(weights["embed"]),
           "lm_head": mat(weights["lm_head"]), "rope": weights["rope"].numpy()}
    for lw in weights["layers"]:
        d = {"attn_norm": vec(lw["attn_norm"]), "mlp_norm": vec(lw["mlp_norm"]),
             "wqkv": mat(lw["wqkv"]), "wo": mat(lw["wo"])}
        if shape.qk_norm:
            d["q_norm"], d["k_norm"] = vec(lw["q_norm"]), vec(lw["k_norm"])
        if shape.n_experts:
            E, Ie, H = shape.n_experts, shape.expert_inter, shape.hidden
            d["router"] = npref.bf16_val(orc.to_np(lw["router"]))
            d["experts_gate_up"] = mat(lw["experts_gate_up"]).reshape(E, 2 * Ie, H)
            d["experts_down"] = mat(lw["experts_down"]).reshape(E, H, Ie)
        else:
            d["w_gate_up"], d["w_down"] = mat(lw["w_gate_up"]), mat(lw["w_down"])
        out["layers"].append(d)
    return out


def _setup(shape, lens, seed=0, num_blocks=64):
    weights = gen.make_weights(shape, seed)
    pool = gen.make_pool(shape, num_blocks)
    alloc = gen.BlockAllocator(num_blocks, seed)
    n = len(lens)
    tables = []
    for r, l in enumerate(lens):
        blocks = alloc.alloc((l + 1 + 15) // 16)
        gen.fill_blocks(pool, blocks, seed, "kv", r)
        tables.append(blocks)
    mb = max(len(t) for t in tables)
    bt = np.zeros((n, mb), dtype=np.int32)
    for r, t in enumerate(tables):
        bt[r, :len(t)] = t
    rng = np.random.default_rng(seed + 100)
    toks = rng.integers(0, shape.vocab, size=n).astype(np.int32)
    return weights, orc.to_np(pool).copy(), bt, toks


def _contig_kv(shape, pool, bt, lens):
    kv = []
    for r, l in enumerate(lens):
        per_layer = []
        for layer in range(shape.n_layers):
            ks, vs = [], []
            for h in range(shape.n_kv_heads):
                k, v = orc.kv_gather(pool, shape.n_kv_heads, 16, 128, layer, h, bt[r], l)
                ks.append(npref.bf16_val(k))
                vs.append(npref.bf16_val(v))
            per_layer.append((np.stack(ks, 1).reshape(l, shape.n_kv_heads, 128),
                              np.stack(vs, 1).reshape(l, shape.n_kv_heads, 128)))
        kv.append(per_layer)
    return kv


CASES = [
    shapes.toy("toy-qknorm"),
    shapes.toy("toy-llama", qk_norm=0, tie_embeddings=1, rms_eps=1e-5, n_q_heads=3, n_kv_heads=1, rope_base=5e5),
    shapes.toy("toy-moe", mlp_inter=0, n_experts=8, top_k=2, expert_inter=64, norm_topk_prob=1),
    shapes.toy("toy-moe-nonorm", mlp_inter=0, n_experts=4, top_k=3, expert_inter=64, norm_topk_prob=0, n_layers=1),
]


@pytest.mark.parametrize("shape", CASES, ids=lambda s: s.name)
def test_whole_step_equals_numpy_restatement(shape):
    lens = [0, 5, 16, 33]
    weights, pool, bt, toks = _setup(shape, lens, seed=1)
    om = orc.OracleModel(shape, weights)
    kv = _contig_kv(shape, pool, bt, lens)
    nxt, logits, taps = om.decode_step(pool, 16, lens, toks, bt, want_taps=True)
    W = _dense_dict(shape, weights)
    rn, rl, rkv, rtaps = npref.decode_step(shape, W, kv, lens, toks)
    assert np.array_equal(npref.bf16_val(taps), rtaps)
    assert np.allclose(logits, rl, rtol=0, atol=1e-6 * np.abs(rl).max())
    assert np.array_equal(nxt, rn)
    # the new token's K, V landed at slot lens[r] of the request's blocks
    for r, l in enumerate(lens):
        for layer in range(shape.n_layers):
            for h in range(shape.n_kv_heads):
                k, v = orc.kv_gather(pool, shape.n_kv_heads, 16, 128, layer, h, bt[r], l + 1)
                assert np.array_equal(npref.bf16_val(k[l]), rkv[r][layer][0][h])
                assert np.array_equal(npref.bf16_val(v[l]), rkv[r][layer][1][h])
                assert np.array_equal(npref.bf16_val(k[:l]), kv[r][layer][0][:, h])   # old tokens untouched


def test_batch_invariance_is_bit_exact():
    shape = shapes.toy("toy-batch", vocab=1024)
    lens = [3, 40, 17, 64, 9, 31, 1, 0, 22, 50, 12, 47, 8, 63, 15, 16]
    weights, pool, bt, toks = _setup(shape, lens, seed=2, num_blocks=96)
    om = orc.OracleModel(shape, weights)
    p_all = pool.copy()
    nxt, logits, taps = om.decode_step(p_all, 16, lens, toks, bt, want_taps=True)
    for r in (0, 7, 15):
        p1 = pool.copy()
        n1, l1, t1 = om.decode_step(p1, 16, [lens[r]], toks[r:r + 1], bt[r:r + 1], want_taps=True)
        assert n1[0] == nxt[r]
        assert np.array_equal(l1[0], logits[r])
        assert np.array_equal(t1[:, 0], taps[:, r])
    # order within the batch does not matter either
    perm = np.random.default_rng(3).permutation(16)
    p2 = pool.copy()
    n2, l2, _ = om.decode_step(p2, 16, np.array(lens)[perm], toks[perm], bt[perm])
    assert np.array_equal(l2, logits[perm])
    assert np.array_equal(p2, p_all)


def test_physical_block_permutation_does_not_change_the_step():
    shape = shapes.toy("toy-perm")
    lens = [20, 35]
    weights, pool, bt, toks = _setup(shape, lens, seed=4, num_blocks=16)
    om = orc.OracleModel(shape, weights)
    perm = np.random.default_rng(5).permutation(16)
    pool_b = np.empty_like(pool)
    pool_b[:, :, perm] = pool
    bt_b = perm[bt].astype(np.int32)
    a = om.decode_step(pool, 16, lens, toks, bt)
    b = om.decode_step(pool_b, 16, lens, toks, bt_b)
    assert np.array_equal(a[1], b[1])
    assert np.array_equal(pool_b[:, :, perm], pool)


def test_layer_limit_runs_a_prefix_of_the_layers():
    shape = shapes.toy("toy-limit", n_layers=3)
    lens = [10]
    weights, pool, bt, toks = _setup(shape, lens, seed=6)
    om = orc.OracleModel(shape, weights)
    _, _, full = om.decode_step(pool.copy(), 16, lens, toks, bt, want_taps=True)
    _, _, part = om.decode_step(pool.copy(), 16, lens, toks, bt, layer_limit=2, want_taps=True)
    assert np.array_equal(part[:3], full[:3]) and np.all(part[3] == 0)


def test_moe_with_one_expert_equals_dense_mlp():
    dense = shapes.toy("toy-e1", n_layers=1)
    moe = dense.with_(mlp_inter=0, n_experts=1, top_k=1, expert_inter=256, norm_topk_prob=1)
    lens = [12, 3]
    weights, pool, bt, toks = _setup(dense, lens, seed=7)
    wm = {**weights, "layers": [dict(lw) for lw in weights["layers"]]}
    for lw in wm["layers"]:
        lw["experts_gate_up"], lw["experts_down"] = lw.pop("w_gate_up"), lw.pop("w_down")
        lw["router"] = torch.zeros(1, dense.hidden, dtype=torch.bfloat16)
    a = orc.OracleModel(dense, weights).decode_step(pool.copy(), 16, lens, toks, bt)
    b = orc.OracleModel(moe, wm).decode_step(pool.copy(), 16, lens, toks, bt)
    assert np.array_equal(a[1], b[1])


def test_moe_expert_relabelling_changes_nothing():
    shape = shapes.toy("toy-relabel", mlp_inter=0, n_experts=8, top_k=2, expert_inter=64, norm_topk_prob=1, n_layers=1)
    lens = [9, 21]
    weights, pool, bt, toks = _setup(shape, lens, seed=8)
    perm = np.random.default_rng(9).permutation(8)
    E, Ie, H = 8, 64, shape.hidden
    wp = {**weights, "layers": [dict(lw) for lw in weights["layers"]]}
    for lw in wp["layers"]:
        lw["router"] = lw["router"][perm]
        lw["experts_gate_up"] = tuple(t.view(E, 2 * Ie, -1)[perm].reshape(E * 2 * Ie, -1) for t in lw["experts_gate_up"])
        lw["experts_down"] = tuple(t.view(E, H, -1)[perm].reshape(E * H, -1) for t in lw["experts_down"])
    a = orc.OracleModel(shape, weights).decode_step(pool.copy(), 16, lens, toks, bt)
    b = orc.OracleModel(shape, wp).decode_step(pool.copy(), 16, lens, toks, bt)
    assert np.array_equal(a[1], b[1])


def test_step_rejects_bad_arguments():
    shape = shapes.toy("toy-bad", n_layers=1)
    weights, pool, bt, toks = _setup(shape, [5], seed=9)
    om = orc.OracleModel(shape, weights)
    with pytest.raises(RuntimeError):
        om.decode_step(pool, 16, [5], [shape.vocab], bt)
    with pytest.raises(RuntimeError):
        om.decode_step(pool, 16, [bt.shape[1] * 16], toks, bt)
