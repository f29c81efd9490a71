"""GPU sampling (q4d_sample, q4d_decode_step_sampled) against the oracle's rule.

The kernel forms its weights with fp32 exp, the oracle with fp64: the weights differ by parts in 10^7, so a draw that
lands within that distance of a boundary between two tokens (or of the top-p cut) may legitimately resolve to the
neighbour.  A GPU token is therefore accepted when it is the oracle's, or when the oracle's own target t lies within
1e-5 of the total weight of that token's interval in the oracle's cumulative order; nearly all draws must match
exactly.
"""
import numpy as np
import pytest
import torch

from gpu_util import Scenario
from oracle import q4d_oracle as orc
from workload import shapes

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def q4d():
    from paper_2601_19139_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def _accept(logits, T, k, p, u, got):
    """(exact, valid) for one request."""
    want = orc.sample_token(logits, T, k, p, u)
    if got == want:
        return True, True
    if not T > 0.0:
        return False, False
    order, w, kept = orc.sampling_table(logits, T, k, p)
    W = int(w[:kept].sum())
    t = min(int(float(np.float32(u)) * float(W)), W - 1)
    pos = int(np.flatnonzero(order == got)[0])
    cum = np.cumsum(w.astype(np.float64))
    lo, hi = (cum[pos - 1] if pos else 0.0), cum[pos]
    tol = 1e-5 * W
    return False, bool(lo - tol <= t <= hi + tol and pos < kept + 1)


def _tables_after(sc, steps):
    """Block tables that cover `steps` more tokens per request (the scenario's own lengths are left alone)."""
    saved = list(sc.lens)
    sc.lens = [l + steps for l in saved]
    bt = sc.block_tables()
    sc.lens = saved
    return bt


CASES = [
    # vocab, temperature, top_k, top_p
    (151936, 1.0, 0, 1.0), (151936, 0.7, 50, 0.9), (151936, 1.5, 0, 0.8), (128256, 0.3, 1000, 1.0),
    (151936, 1.0, 1, 1.0), (151936, 0.0, 40, 0.5), (5000, 2.0, 4999, 0.999), (33, 1.0, 5, 0.5), (1000, 0.05, 0, 0.3),
]


@pytest.mark.parametrize("V,T,k,p", CASES)
def test_sample_matches_the_oracle_rule(q4d, V, T, k, p):
    rng = np.random.default_rng(V + k)
    n = 16
    logits = (rng.standard_normal((n, V)) * rng.uniform(1.0, 5.0, size=(n, 1))).astype(np.float32)
    us = rng.uniform(0, 1, size=n).astype(np.float32)
    us[0], us[1] = 0.0, np.float32(1.0 - 2.0 ** -24)
    got = q4d.sample(torch.from_numpy(logits).cuda(), [T] * n, [k] * n, [p] * n, us).cpu().numpy()
    exact = 0
    for r in range(n):
        e, ok = _accept(logits[r], T, k, p, float(us[r]), int(got[r]))
        assert ok, (r, int(got[r]), orc.sample_token(logits[r], T, k, p, float(us[r])))
        exact += e
    assert exact >= n - 1


def test_sample_with_planted_ties_and_mixed_settings(q4d):
    """Equal logits (the position among them is decided in index order), a different setting per request, greedy and
    sampled requests in one call."""
    rng = np.random.default_rng(9)
    V, n = 20000, 16
    logits = (rng.standard_normal((n, V)) * 2.0).astype(np.float32)
    for r in range(n):
        logits[r, rng.integers(0, V, size=4000)] = logits[r, int(rng.integers(0, V))]   # thousands of equal logits
        logits[r, rng.integers(0, V, size=3)] = logits[r].max()                          # and a tie for the largest
    T = rng.choice([0.0, 0.5, 1.0, 3.0], size=n).astype(np.float32)
    k = rng.choice([0, 1, 10, 5000, V], size=n).astype(np.int32)
    p = rng.choice([1.0, 0.9, 0.2], size=n).astype(np.float32)
    us = rng.uniform(0, 1, size=n).astype(np.float32)
    got = q4d.sample(torch.from_numpy(logits).cuda(), T, k, p, us).cpu().numpy()
    exact = 0
    for r in range(n):
        e, ok = _accept(logits[r], float(T[r]), int(k[r]), float(p[r]), float(us[r]), int(got[r]))
        assert ok, (r, float(T[r]), int(k[r]), float(p[r]))
        exact += e
    assert exact >= n - 1


def test_sampled_frequencies_follow_the_softmax(q4d):
    """2048 draws on an even grid of u from one small distribution: the frequencies are the probabilities."""
    rng = np.random.default_rng(10)
    V = 64
    l = (rng.standard_normal(V) * 1.5).astype(np.float32)
    counts = np.zeros(V)
    grid = (np.arange(2048) + 0.5) / 2048
    lt = torch.from_numpy(np.tile(l, (16, 1))).cuda()
    for i in range(0, 2048, 16):
        us = grid[i:i + 16].astype(np.float32)
        counts += np.bincount(q4d.sample(lt, [1.0] * 16, [0] * 16, [1.0] * 16, us).cpu().numpy(), minlength=V)
    prob = np.exp(l.astype(np.float64) - l.max())
    prob /= prob.sum()
    assert np.abs(counts / 2048 - prob).max() <= 1.5 / 2048


def test_decode_step_sampled_draws_from_the_steps_logits(q4d):
    shape = shapes.toy("gpu-toy-sampled", hidden=256, n_q_heads=4, n_kv_heads=2, mlp_inter=512, vocab=1024)
    sc = Scenario(shape, [10, 31, 47], seed=21)
    model = q4d.Model(shape, sc.weights)
    pool = q4d.KVPool(model, sc.pool)
    ids = np.arange(3, dtype=np.int64)
    for r in range(3):
        pool.request_admit(r, sc.lens[r])
    nxt = torch.zeros(3, dtype=torch.int32, device="cuda")
    lg = torch.zeros(3, shape.vocab, dtype=torch.float32, device="cuda")
    T, k, p, us = [0.0, 1.0, 0.8], [0, 20, 0], [1.0, 1.0, 0.7], np.array([0.3, 0.6, 0.9], dtype=np.float32)
    q4d.decode_step_sampled(model, pool, ids, sc.tokens, sc.block_tables(), T, k, p, us, nxt, lg)
    torch.cuda.synchronize()
    g = lg.cpu().numpy()
    got = nxt.cpu().numpy()
    for r in range(3):      # the draw is judged on the logits the step produced
        _, ok = _accept(g[r], T[r], k[r], p[r], float(us[r]), int(got[r]))
        assert ok, r
    assert got[0] == int(g[0].argmax())
    assert pool.request_len(0) == 11
    # without a logits buffer the step draws from its workspace copy
    q4d.decode_step_sampled(model, pool, ids, sc.tokens, _tables_after(sc, 1), T, k, p, us, nxt)
    torch.cuda.synchronize()
    assert pool.request_len(0) == 12
    with pytest.raises(q4d.Q4dError) as ei:
        q4d.decode_step_sampled(model, pool, ids, sc.tokens, _tables_after(sc, 2), T, k, p, [0.1, 1.0, 0.2], nxt)
    assert ei.value.code == -1 and pool.request_len(0) == 12
    pool.close()
    model.close()
