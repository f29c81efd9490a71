"""Oracles of the two caches of the paper's serving loop, written from the printed algorithms.

TEST INFRASTRUCTURE ONLY (tests import it; the CUDA library never does and shares nothing with it).

Text prefix cache: Algorithm 2 ("Text Prefix Cache Lookup") exactly as printed: hash the whole prompt, then every
shorter prefix from |P| down to 1, return the first entry found and the length it covers.  SHA-256 is the library
routine (hashlib).  What the algorithm leaves open, and the reading taken (all listed in the design doc):
  * what gets stored: after a prompt has been processed, an entry for every 16-token-aligned prefix of it (key: the
    SHA-256 of that prefix's int32 token ids), whose KV state is the list of pool blocks holding those tokens; a key
    that is already present keeps its entry (and its blocks);
  * recency: a hit on a prefix is a use of it and of every stored prefix of it (their KV state is part of the hit);
  * eviction (Section 3.3: LRU within a byte budget, 512 MB by default): the least recently used entry that no
    request is reading and that is not a proper prefix of another stored entry, repeated until the budget holds.

Multimodal store: Algorithm 3 ("Cache-Aware Multimodal Generation"): key = SHA-256 of the decoded pixel bytes, value
= (embeddings, KV state); same LRU budget; an entry in use is never evicted.
"""
import hashlib

import numpy as np

BLOCK = 16
DEFAULT_CAPACITY = 512 << 20


def _h(tokens):
    return hashlib.sha256(np.asarray(tokens, dtype="<i4").tobytes()).digest()


class PrefixCacheOracle:
    def __init__(self, capacity_bytes, bytes_per_block):
        self.capacity = capacity_bytes or DEFAULT_CAPACITY
        self.bytes_per_block = bytes_per_block
        self.C = {}      # hash -> {"tokens": tuple, "blocks": list, "readers": int, "last_use": int}
        self.clock = 0

    def lookup(self, P):
        """Algorithm 2.  Returns (kv_state as a list of blocks, start position); readers of the hit are counted."""
        P = list(P)
        h = _h(P)
        if h in self.C:                                   # full cache hit
            return self._hit(self.C[h]), len(P)
        for i in range(len(P), 0, -1):                    # i = |P| down to 1
            ph = _h(P[:i])
            if ph in self.C:
                return self._hit(self.C[ph]), i           # partial hit
        return [], 0                                      # cache miss

    def _hit(self, entry):
        toks = entry["tokens"]
        for n in range(BLOCK, len(toks) + 1, BLOCK):      # the entry and every stored prefix of it, shortest first
            e = self.C[_h(toks[:n])]
            e["readers"] += 1
            self.clock += 1
            e["last_use"] = self.clock
        return list(entry["blocks"])

    def insert(self, P, block_table):
        """Store every block-aligned prefix of the processed prompt (the inserting request reads what it adds).
        Returns, per full block, whether the cache holds exactly that block for that prefix afterwards;
        self.last_created lists the prefix lengths (in blocks) this call added."""
        P = list(P)
        adopted, created = [], []
        chain = []
        for n in range(BLOCK, (min(len(P) // BLOCK, len(block_table))) * BLOCK + 1, BLOCK):
            key = _h(P[:n])
            self.clock += 1
            if key in self.C:
                e = self.C[key]
                e["last_use"] = self.clock
                adopted.append(1 if e["blocks"][-1] == block_table[n // BLOCK - 1] else 0)
                chain = list(e["blocks"])
                continue
            chain = chain + [int(block_table[n // BLOCK - 1])]
            self.C[key] = {"tokens": tuple(P[:n]), "blocks": list(chain), "readers": 1, "last_use": self.clock}
            adopted.append(1)
            created.append(n // BLOCK)
        self.last_created = created
        return adopted

    def release(self, P, block_counts):
        """A request stops reading the prefixes of P with the given lengths in blocks (those a lookup returned to it
        or its insert created)."""
        for nb in block_counts:
            self.C[_h(list(P)[:nb * BLOCK])]["readers"] -= 1

    def evict(self, bytes_to_free=0):
        held = len(self.C) * self.bytes_per_block
        target = max(held - self.capacity, 0, bytes_to_free)
        freed, out = 0, []
        while freed < target:
            cands = []
            for k, e in self.C.items():
                if e["readers"]:
                    continue
                t = e["tokens"]
                if any(len(o["tokens"]) > len(t) and o["tokens"][:len(t)] == t for o in self.C.values()):
                    continue                              # a longer stored prefix builds on it
                cands.append((e["last_use"], k))
            if not cands:
                break
            _, k = min(cands)
            out.append(self.C[k]["blocks"][-1])
            del self.C[k]
            freed += self.bytes_per_block
        return out


class ContentCacheOracle:
    """Algorithm 3's Cache: hash of the pixel bytes -> (embeddings, kv_state), LRU within a byte budget."""

    def __init__(self, capacity_bytes):
        self.capacity = capacity_bytes or DEFAULT_CAPACITY
        self.cache = {}
        self.clock = 0

    def lookup(self, pixels):
        h = hashlib.sha256(pixels).digest()
        if h in self.cache:
            e = self.cache[h]
            e["readers"] += 1
            self.clock += 1
            e["last_use"] = self.clock
            return True, h, e
        return False, h, None

    def store(self, h, embeddings, kv_state, n_tokens, nbytes):
        assert h not in self.cache
        self.clock += 1
        self.cache[h] = {"embeddings": embeddings, "kv_state": list(kv_state), "n_tokens": n_tokens, "bytes": nbytes,
                         "readers": 1, "last_use": self.clock}

    def release(self, h):
        self.cache[h]["readers"] -= 1

    def evict(self, bytes_to_free=0):
        gone = []
        while sum(e["bytes"] for e in self.cache.values()) > self.capacity or bytes_to_free > 0:
            cands = [(e["last_use"], h) for h, e in self.cache.items() if not e["readers"]]
            if not cands:
                break
            _, h = min(cands)
            gone.append((h, self.cache[h]))
            bytes_to_free = max(0, bytes_to_free - self.cache[h]["bytes"])
            del self.cache[h]
        return gone
