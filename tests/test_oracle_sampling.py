"""Pins of the oracle's sampling rule (oracle.q4d_oracle.sample_token) against what the mathematics fixes."""
import numpy as np

from oracle import q4d_oracle as orc


def _logits(V, seed, scale=3.0):
    return (np.random.default_rng(seed).standard_normal(V) * scale).astype(np.float32)


def _brute(logits, T, k, p, u):
    """The same rule spelt with Python lists and loops (sorted(), a running sum)."""
    V = len(logits)
    idx = sorted(range(V), key=lambda j: (-float(logits[j]), j))
    m = float(logits[idx[0]])
    w = [int(np.rint(np.exp((float(logits[j]) - m) / T) * 2.0 ** 40)) for j in idx]
    kept = V
    if 0 < k < V:
        kth = float(logits[idx[k - 1]])
        kept = sum(1 for j in idx if float(logits[j]) >= kth)
    if p < 1.0:
        Wk = sum(w[:kept])
        target = min(max(int(np.ceil(float(np.float32(p)) * float(Wk))), 1), Wk)
        run = 0
        for pos in range(kept):
            run += w[pos]
            if run >= target:
                c = float(logits[idx[pos]])
                break
        kept = min(kept, sum(1 for j in idx if float(logits[j]) >= c))
    W = sum(w[:kept])
    t = min(int(float(np.float32(u)) * float(W)), W - 1)
    run = 0
    for pos in range(kept):
        run += w[pos]
        if run > t:
            return idx[pos]
    raise AssertionError("unreachable")


def test_temperature_zero_and_tiny_temperature_are_greedy():
    l = _logits(500, 0)
    l[[17, 230]] = l.max() + 1.0                       # a tie for the largest: the lower index wins
    assert orc.sample_token(l, 0.0, 0, 1.0, 0.73) == 17
    l2 = _logits(500, 1)
    for u in (0.0, 0.31, 0.999999):
        assert orc.sample_token(l2, 1e-4, 0, 1.0, u) == int(l2.argmax())


def test_top_k_one_is_greedy_and_ties_at_the_cut_stay():
    l = _logits(300, 2)
    for u in (0.0, 0.5, 0.99):
        assert orc.sample_token(l, 1.0, 1, 1.0, u) == int(l.argmax())
    l = np.array([0.0, 2.0, 1.0, 1.0, -1.0, 1.0], dtype=np.float32)
    order, w, kept = orc.sampling_table(l, 1.0, 2, 1.0)
    assert kept == 4 and list(order[:4]) == [1, 2, 3, 5]          # the second largest value is held by three tokens
    drawn = {orc.sample_token(l, 1.0, 2, 1.0, u) for u in np.linspace(0, 0.9999, 400)}
    assert drawn == {1, 2, 3, 5}


def test_plain_categorical_frequencies_follow_the_softmax():
    l = _logits(40, 3, 1.5)
    T = 0.8
    us = (np.arange(20000) + 0.5) / 20000                 # an even grid of draws: frequencies = interval lengths
    counts = np.bincount([orc.sample_token(l, T, 0, 1.0, u) for u in us], minlength=40) / us.size
    p = np.exp((l.astype(np.float64) - l.max()) / T)
    p /= p.sum()
    assert np.abs(counts - p).max() <= 1.0 / us.size + 1e-9


def test_top_p_keeps_the_smallest_set_that_reaches_the_mass():
    l = _logits(200, 4)
    T, p_cut = 1.3, 0.6
    order, w, kept = orc.sampling_table(l, T, 0, p_cut)
    prob = w / w.sum()
    assert prob[:kept].sum() >= p_cut - 1e-9
    assert prob[:kept - 1].sum() < p_cut                   # distinct logits here: one fewer falls short
    drawn = {orc.sample_token(l, T, 0, p_cut, u) for u in np.linspace(0, 0.99999, 3000)}
    assert drawn == set(int(j) for j in order[:kept])
    # inside the kept set the frequencies are the renormalised probabilities
    us = (np.arange(30000) + 0.5) / 30000
    counts = np.bincount([orc.sample_token(l, T, 0, p_cut, u) for u in us], minlength=200) / us.size
    want = np.zeros(200)
    want[order[:kept]] = prob[:kept] / prob[:kept].sum()
    assert np.abs(counts - want).max() <= 1.0 / us.size + 1e-9


def test_rank_of_the_drawn_token_is_monotone_in_u():
    l = _logits(1000, 5)
    order, _, _ = orc.sampling_table(l, 1.0, 50, 0.9)
    rank = {int(j): i for i, j in enumerate(order)}
    ranks = [rank[orc.sample_token(l, 1.0, 50, 0.9, u)] for u in np.linspace(0, 0.99999, 500)]
    assert all(a <= b for a, b in zip(ranks, ranks[1:]))


def test_against_the_rule_spelt_with_loops():
    rng = np.random.default_rng(6)
    for case in range(60):
        V = int(rng.integers(2, 400))
        l = _logits(V, 100 + case, float(rng.uniform(0.5, 6.0)))
        if case % 3 == 0:                                   # planted ties
            l[rng.integers(0, V, size=V // 2)] = l[int(rng.integers(0, V))]
        T = float(rng.uniform(0.2, 2.0))
        k = int(rng.choice([0, 1, 2, V // 2, V, V + 5]))
        p = float(rng.choice([1.0, 0.95, 0.5, 0.1]))
        u = float(rng.uniform(0, 1))
        assert orc.sample_token(l, T, k, p, u) == _brute(l, T, k, p, u), (case, V, T, k, p, u)
