"""The host-side caches of the library against the printed algorithms (oracle/cache_oracle.py), and the pins of
those oracles: SHA-256 against its published test vectors, Algorithm 2's worst case (every prefix length tried),
LRU order and the byte budget by hand-worked sequences."""
import hashlib

import numpy as np
import pytest

from oracle.cache_oracle import ContentCacheOracle, PrefixCacheOracle


@pytest.fixture(scope="module")
def q4d():
    from paper_2601_19139_b200 import binding, build
    build.build()
    binding.lib()
    return binding


# ---- SHA-256 ---------------------------------------------------------------------------

def test_sha256_matches_the_published_vectors_and_the_library_routine(q4d):
    # FIPS 180-4 examples: "abc" and the 448-bit message; the empty string
    assert q4d.sha256(b"abc").hex() == "ba7816bf8f01cfea414140de5dae2223b00361a396177a9cb410ff61f20015ad"
    assert q4d.sha256(b"abcdbcdecdefdefgefghfghighijhijkijkljklmklmnlmnomnopnopq").hex() == \
        "248d6a61d20638b8e5c026930c3e6039a33ce45964ff2167f6ecedd419db06c1"
    assert q4d.sha256(b"").hex() == "e3b0c44298fc1c149afbf4c8996fb92427ae41e4649b934ca495991b7852b855"
    rng = np.random.default_rng(0)
    for n in (1, 55, 56, 63, 64, 65, 119, 120, 1000, 70001):      # around the padding boundaries
        data = rng.integers(0, 256, size=n, dtype=np.uint8).tobytes()
        assert q4d.sha256(data) == hashlib.sha256(data).digest()


# ---- pins of the prefix-cache oracle ---------------------------------------------------

def test_oracle_lookup_is_algorithm_2_on_hand_worked_prompts():
    c = PrefixCacheOracle(0, 100)
    sys_prompt = list(range(1000, 1040))                         # 40 tokens: two full blocks and a tail
    assert c.lookup(sys_prompt) == ([], 0)                       # empty cache: miss, start at 0
    assert c.insert(sys_prompt, [7, 3, 9]) == [1, 1]             # only full blocks are stored
    c.release(sys_prompt, [1, 2])
    assert c.lookup(sys_prompt[:32]) == ([7, 3], 32)             # full hit: the hash of the whole prompt
    c.release(sys_prompt, [1, 2])
    assert c.lookup(sys_prompt) == ([7, 3], 32)                  # partial hit found on the way down from |P| = 40
    c.release(sys_prompt, [1, 2])
    other = sys_prompt[:16] + [5] * 30
    assert c.lookup(other) == ([7], 16)                          # shares only the first block
    c.release(other, [1])
    assert c.lookup([1] + sys_prompt) == ([], 0)                 # same tokens shifted by one: nothing in common


def test_oracle_eviction_is_lru_among_unread_leaves_within_the_budget():
    c = PrefixCacheOracle(3 * 100, 100)                          # room for three blocks
    a, b = list(range(32)), list(range(100, 132))
    c.insert(a, [0, 1]); c.release(a, [1, 2])
    c.insert(b, [2, 3]); c.release(b, [1, 2])
    assert len(c.C) == 4
    assert c.evict() == [1]                                      # over by one: the oldest leaf is a's second block
    c.lookup(a[:16]); c.release(a, [1])                          # a's first block is now the most recent
    assert c.evict(100) == [3]                                   # asked for one more: b's leaf (b's root has a child)
    assert c.evict(200) == [2, 0]
    c.insert(a, [4, 5])                                          # still read by the inserting request
    assert c.evict(10 ** 9) == []


# ---- library against the oracle --------------------------------------------------------

def _prompts(rng, count):
    """Prompts with shared system prefixes of several lengths, exact repeats and unrelated ones."""
    systems = [rng.integers(0, 50000, size=int(n)).tolist() for n in (16, 48, 100, 512)]
    out = []
    for _ in range(count):
        kind = rng.integers(0, 4)
        if kind == 0:
            p = rng.integers(0, 50000, size=int(rng.integers(1, 200))).tolist()
        elif kind == 3 and out:
            p = list(out[int(rng.integers(0, len(out)))])
        else:
            s = systems[int(rng.integers(0, len(systems)))]
            p = s[:int(rng.integers(1, len(s) + 1))] + rng.integers(0, 50000, size=int(rng.integers(0, 120))).tolist()
        out.append(p)
    return out


@pytest.mark.parametrize("capacity_blocks", [10 ** 6, 40])
def test_prefix_cache_equals_algorithm_2_on_seeded_prompt_streams(q4d, capacity_blocks):
    """Every request: look up, allocate the missing blocks, insert, and (a few requests later) release; with the
    small budget the cache evicts after every request.  Hit length, block list, adoption flags, evicted blocks and
    entry count must be identical to the oracle's at every step."""
    rng = np.random.default_rng(capacity_blocks)
    bpb = 4096
    lib_c = q4d.PrefixCache(capacity_blocks * bpb, bpb)
    orc_c = PrefixCacheOracle(capacity_blocks * bpb, bpb)
    next_block = 0
    active = []
    hits = 0
    for step, P in enumerate(_prompts(rng, 300)):
        blocks, handles = lib_c.lookup(P)
        o_blocks, o_start = orc_c.lookup(P)
        assert blocks == o_blocks and 16 * len(blocks) == o_start, (step, len(P))
        hits += len(blocks)
        table = list(blocks)
        while len(table) < (len(P) + 15) // 16:
            table.append(next_block)
            next_block += 1
        new_handles, adopted = lib_c.insert(P, table)
        assert adopted == orc_c.insert(P, table), step
        created = [i + 1 for i, h in enumerate(new_handles) if h >= 0]
        assert created == orc_c.last_created, step
        active.append((P, handles + [h for h in new_handles if h >= 0], list(range(1, len(blocks) + 1)) + created))
        if len(active) > 3:                               # an older request finishes
            Pd, hd, counts = active.pop(int(rng.integers(0, len(active))))
            lib_c.release(hd)
            orc_c.release(Pd, counts)
        assert lib_c.evict() == orc_c.evict(), step
        assert lib_c.stats()["entries"] == len(orc_c.C)
    assert hits > 100                                     # the stream does share prefixes
    assert lib_c.stats()["hit_blocks"] == hits and lib_c.stats()["lookups"] == 300
    lib_c.close()


def test_prefix_cache_worst_case_every_prefix_length_is_tried(q4d):
    """A 512-token prompt whose first 496 tokens are cached, then prompts that diverge at every possible position:
    Algorithm 2 walks down through every prefix length; the block-chained lookup must land on the same length."""
    rng = np.random.default_rng(5)
    base = rng.integers(0, 50000, size=512).tolist()
    lib_c, orc_c = q4d.PrefixCache(0, 1), PrefixCacheOracle(0, 1)
    table = list(range(100, 132))
    assert lib_c.insert(base[:496], table)[1] == orc_c.insert(base[:496], table) == [1] * 31
    for cut in list(range(0, 513, 7)) + [15, 16, 17, 495, 496, 497, 512]:
        P = base[:cut] + [60000 + cut] * (512 - cut)      # identical up to `cut`, different afterwards
        blocks, handles = lib_c.lookup(P)
        o_blocks, o_start = orc_c.lookup(P)
        assert (blocks, 16 * len(blocks)) == (o_blocks, o_start)
        assert o_start == min(cut, 496) // 16 * 16
        lib_c.release(handles)
        orc_c.release(P, range(1, len(blocks) + 1))
    lib_c.close()


def test_prefix_cache_rejects_bad_calls(q4d):
    c = q4d.PrefixCache(0, 64)
    with pytest.raises(q4d.Q4dError):
        c.release([5])                                    # a handle nobody holds
    assert c.lookup([]) == ([], []) and c.evict() == []
    assert c.stats() == {"entries": 0, "bytes": 0, "lookups": 1, "hit_blocks": 0}
    c.close()
    with pytest.raises(q4d.Q4dError):
        q4d.PrefixCache(0, 0)


# ---- content-hash store (Algorithm 3) --------------------------------------------------

def test_content_cache_equals_algorithm_3_store_on_a_seeded_image_stream(q4d):
    """Images arrive repeatedly (the same pixels, however they were delivered, hash alike); a miss stores embeddings
    and KV state, a hit returns them; the byte budget evicts least recently used entries that nobody is using."""
    rng = np.random.default_rng(11)
    images = [rng.integers(0, 256, size=int(rng.integers(100, 5000)), dtype=np.uint8).tobytes() for _ in range(12)]
    cap = 40000
    lib_c, orc_c = q4d.ContentCache(cap), ContentCacheOracle(cap)
    in_use = []
    next_block, hits = 0, 0
    for step in range(200):
        px = images[int(rng.integers(0, len(images)))]
        hit, entry, blocks = lib_c.lookup(bytes(px))
        o_hit, h, o_e = orc_c.lookup(px)
        assert hit == o_hit and bytes(entry.hash) == h == __import__("hashlib").sha256(px).digest()
        if hit:
            hits += 1
            assert blocks == o_e["kv_state"] and entry.embeddings == o_e["embeddings"] and entry.n_tokens == o_e["n_tokens"]
        else:                                              # "VisionEncoder" ran: store its result (Algorithm 3)
            nb = int(rng.integers(1, 6))
            blocks = list(range(next_block, next_block + nb))
            next_block += nb
            entry.embeddings, entry.bytes, entry.n_tokens = 0x1000 + step, len(px) * 3, nb * 16
            lib_c.store(entry, blocks)
            orc_c.store(h, 0x1000 + step, blocks, nb * 16, len(px) * 3)
        in_use.append(h)
        if len(in_use) > 2:
            done = in_use.pop(0)
            lib_c.release(done)
            orc_c.release(done)
        gone = lib_c.evict()
        o_gone = orc_c.evict()
        assert [(bytes(e.hash), b) for e, b in gone] == [(hh, e["kv_state"]) for hh, e in o_gone], step
        st = lib_c.stats()
        assert st["entries"] == len(orc_c.cache) and st["bytes"] == sum(e["bytes"] for e in orc_c.cache.values())
    assert hits > 50
    lib_c.close()


def test_content_cache_hand_worked_lru():
    c = ContentCacheOracle(100)
    for name, size in ((b"a", 40), (b"b", 40), (b"c", 40)):
        _, h, _ = c.lookup(name)
        c.store(h, name, [], 0, size)
        c.release(h)
    assert [e["embeddings"] for _, e in c.evict()] == [b"a"]      # 120 > 100: the oldest goes
    c.lookup(b"b")                                                 # b is in use and most recent
    _, h, _ = c.lookup(b"d")
    c.store(h, b"d", [], 0, 60)
    c.release(h)
    assert [e["embeddings"] for _, e in c.evict()] == [b"c"]      # 140 > 100: c is the oldest unused; then 100 fits
    assert sorted(e["embeddings"] for e in c.cache.values()) == [b"b", b"d"]
