"""Prompt processing (q4d_prefill): pins of the oracle's definition on the CPU, GPU parity against it."""
import numpy as np
import pytest
import torch

from oracle import q4d_oracle as orc
from workload import gen, shapes


def _toy():
    return shapes.toy("prefill-toy", n_layers=2, hidden=256, n_q_heads=4, n_kv_heads=2, mlp_inter=512, vocab=1024)


def _setup(shape, seed, n_blocks, device="cpu"):
    weights = gen.make_weights(shape, seed, device)
    pool_t = gen.make_pool(shape, n_blocks, device)
    return weights, pool_t


def test_oracle_prefill_is_causal_and_resumes_from_any_cached_prefix():
    """What the definition implies: K, V of a position depend on the tokens up to it and on nothing after; resuming
    after a cached prefix gives bit-identical K, V and logits to processing the whole prompt."""
    shape = _toy()
    weights, pool_t = _setup(shape, 1, 16)
    om = orc.OracleModel(shape, weights)
    rng = np.random.default_rng(2)
    prompt = rng.integers(0, shape.vocab, size=45).astype(np.int32)
    table = [9, 2, 11, 5]
    full = orc.to_np(pool_t).copy()
    nxt_full, lg_full = orc.prefill(om, full, 16, prompt, 0, table)
    # causal: a different tail leaves the K, V of the common prefix untouched
    other = prompt.copy()
    other[30:] = rng.integers(0, shape.vocab, size=15)
    alt = orc.to_np(pool_t).copy()
    orc.prefill(om, alt, 16, other, 0, table)
    for blk, upto in ((9, 16), (2, 14)):                      # tokens 0..15 and 16..29
        assert np.array_equal(full[:, :, blk, :, :upto], alt[:, :, blk, :, :upto])
    assert not np.array_equal(full[:, :, 2, :, 14:], alt[:, :, 2, :, 14:])
    # resuming at 32 over the K, V of the first 32 tokens: the same pool, the same answer
    resumed = orc.to_np(pool_t).copy()
    resumed[:, :, [9, 2]] = full[:, :, [9, 2]]
    nxt_res, lg_res = orc.prefill(om, resumed, 16, prompt, 32, table)
    assert nxt_res == nxt_full and np.array_equal(lg_res, lg_full)
    assert np.array_equal(resumed[:, :, table], full[:, :, table])
    # and the request then decodes as if it had been built token by token
    a, la, _ = om.decode_step(full, 16, [45], [nxt_full], np.array([table], dtype=np.int32))
    b, lb, _ = om.decode_step(resumed, 16, [45], [nxt_res], np.array([table], dtype=np.int32))
    assert a[0] == b[0] and np.array_equal(la, lb)


@pytest.fixture(scope="module")
def q4d():
    from paper_2601_19139_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def _kv_err(got_bits, want_bits):
    g, w = orc.bf16_to_f64(got_bits), orc.bf16_to_f64(want_bits)
    rms = float(np.sqrt((w ** 2).mean()))
    return float(np.abs(g - w).max()) / rms, float(np.sqrt(((g - w) ** 2).mean())) / rms


@pytest.mark.gpu
@pytest.mark.parametrize("shape,n_tokens,start", [
    (_toy(), 45, 0), (_toy(), 16, 0), (_toy(), 1, 0), (_toy(), 70, 32), (_toy(), 33, 32),
    (shapes.toy("prefill-toy-llama", n_layers=2, hidden=512, n_q_heads=6, n_kv_heads=2, mlp_inter=768, vocab=2000,
                qk_norm=0, rms_eps=1e-5, rope_base=5e5), 100, 48),
    (shapes.toy("prefill-toy-moe", n_layers=2, hidden=256, n_q_heads=4, n_kv_heads=2, mlp_inter=256, vocab=1024,
                n_experts=8, top_k=2, expert_inter=256, norm_topk_prob=1), 40, 16),
], ids=lambda v: getattr(v, "name", str(v)))
def test_prefill_matches_the_oracle(q4d, shape, n_tokens, start):
    from gpu_util import bits, from_bits
    weights, pool_t = _setup(shape, 3, 24, "cuda")
    om = orc.OracleModel(shape, weights)
    rng = np.random.default_rng(n_tokens + start)
    prompt = rng.integers(0, shape.vocab, size=n_tokens).astype(np.int32)
    table = [7, 20, 3, 11, 15, 1, 9][:max(1, (n_tokens + 15) // 16)]
    host = orc.to_np(pool_t).copy()
    if start:   # the cached prefix: the oracle's K, V of the first `start` tokens, present on both sides
        orc.prefill(om, host, 16, prompt[:start], 0, table)
        for b in table[:(start + 15) // 16]:
            pool_t[:, :, b] = from_bits(host[:, :, b])
    o_next, o_logits = orc.prefill(om, host, 16, prompt, start, table)
    model = q4d.Model(shape, weights)
    pool = q4d.KVPool(model, pool_t)
    nxt = torch.zeros(1, dtype=torch.int32, device="cuda")
    lg = torch.zeros(shape.vocab, dtype=torch.float32, device="cuda")
    q4d.prefill(model, pool, 42, prompt, start, table, nxt, lg)
    torch.cuda.synchronize()
    assert pool.request_len(42) == n_tokens
    # K, V of the processed tokens, every layer (free-running through two layers: rounding differences only)
    got = bits(pool_t)
    for t in range(start, n_tokens):
        emax, erms = _kv_err(got[:, :, table[t // 16], :, t % 16], host[:, :, table[t // 16], :, t % 16])
        assert erms <= 1e-2 and emax <= 0.15, (t, emax, erms)
    # tokens before start_pos and blocks of other requests are untouched
    if start:
        assert np.array_equal(got[:, :, table[0], :, :min(start, 16)], host[:, :, table[0], :, :min(start, 16)])
    assert np.array_equal(got[:, :, 0], orc.to_np(gen.make_pool(shape, 24, "cpu"))[:, :, 0])
    g = lg.cpu().numpy().astype(np.float64)
    rms = np.sqrt((o_logits.astype(np.float64) ** 2).mean())
    err = np.abs(g - o_logits).max() / rms
    tol = 0.15 if shape.n_experts else 4e-2      # routing is a discontinuous decision (see the step tests)
    assert err <= tol, err
    tok = int(nxt.cpu().numpy()[0])
    assert tok == o_next or o_logits[o_next] - o_logits[tok] <= 2 * err * rms
    # the request continues with ordinary decode steps
    nxt2 = torch.zeros(1, dtype=torch.int32, device="cuda")
    bt = np.array([table + [22]], dtype=np.int32)
    q4d.decode_step(model, pool, np.array([42], dtype=np.int64), np.array([o_next], dtype=np.int32), bt, nxt2)
    torch.cuda.synchronize()
    assert pool.request_len(42) == n_tokens + 1
    pool.close()
    model.close()


@pytest.mark.gpu
def test_prefill_rejects_bad_calls(q4d):
    shape = _toy()
    weights, pool_t = _setup(shape, 4, 8, "cuda")
    model = q4d.Model(shape, weights)
    pool = q4d.KVPool(model, pool_t)
    toks = np.arange(20, dtype=np.int32)
    for args, code in (((toks, 20, [0, 1]), -1), ((toks, 0, [0]), -5), ((toks, 0, [0, 99]), -6),
                       ((np.array([5000], dtype=np.int32), 0, [0]), -1)):
        with pytest.raises(q4d.Q4dError) as ei:
            q4d.prefill(model, pool, 1, *args)
        assert ei.value.code == code
    q4d.prefill(model, pool, 1, toks, 0, [0, 1])
    with pytest.raises(q4d.Q4dError) as ei:
        q4d.prefill(model, pool, 1, toks, 0, [2, 3])
    assert ei.value.code == -3
    pool.close()
    model.close()
