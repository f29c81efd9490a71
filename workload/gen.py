"""Seeded synthetic inputs shared by the CPU oracle and the CUDA library.

Everything here is input preparation: random weights and their 4-bit packing,
norm weights, the rotary table, prefilled KV blocks, block allocation and the
admit/release script of the continuous-batching loop (Algorithm 1 of the
paper).  No step of the decode path is computed here.  All tensors are torch
tensors on the requested device; the same arrays are handed to both sides.

Recipe (stands in for the paper's checkpoints and prompts, which are not
available): projection weights ~ N(0, 0.02) per tensor, quantised per group of
64 input features to 4-bit codes with bf16 scale and bias; norm weights
1 + N(0, 0.02) rounded to bf16; router ~ N(0, 0.02) bf16; prefilled K, V
~ N(0, 1) bf16; first tokens uniform over the vocabulary.
"""
import hashlib
import math

import numpy as np
import torch

BLOCK_SIZE = 16


def _seed(*parts):
    h = hashlib.sha256("/".join(str(p) for p in parts).encode()).digest()
    return int.from_bytes(h[:8], "little") & 0x7FFFFFFFFFFFFFFF


def _gen(device, *parts):
    g = torch.Generator(device=device)
    g.manual_seed(_seed(*parts))
    return g


# ------------------------------------------------------------------ quantiser

def quantize_q4(w):
    """float32 [N][K] -> (codes int32 [N][K/8] (uint32 bit patterns), scales bf16 [N][K/64], biases bf16 [N][K/64]).

    Per group of 64 consecutive input features, in fp32 IEEE arithmetic:
    bias = bf16(min), scale = bf16((max - min) / 15),
    code = clamp(round_half_even((w - bias) / scale), 0, 15); a group whose scale
    rounds to zero takes scale 1 and code 0.  Element k of a row sits in word
    k >> 3 at bits 4*(k & 7).. (lowest nibble first).
    """
    assert w.dtype == torch.float32 and w.dim() == 2 and w.shape[1] % 64 == 0
    N, K = w.shape
    g = w.view(N, K // 64, 64)
    lo, hi = g.amin(-1), g.amax(-1)
    fifteen = torch.full((), 15.0, dtype=torch.float32, device=w.device)
    bias = lo.to(torch.bfloat16)
    scale = torch.div(hi - lo, fifteen).to(torch.bfloat16)
    flat = ~(scale.float() > 0)
    scale = torch.where(flat, torch.ones_like(scale), scale)
    t = torch.div(g - bias.float().unsqueeze(-1), scale.float().unsqueeze(-1))
    code = torch.round(t).clamp_(0, 15)
    code = torch.where(flat.unsqueeze(-1), torch.zeros_like(code), code).to(torch.int64)
    code = code.view(N, K // 8, 8)
    shifts = torch.arange(8, device=w.device, dtype=torch.int64) * 4
    word = (code << shifts).sum(-1)
    word = torch.where(word >= 2 ** 31, word - 2 ** 32, word).to(torch.int32)
    return word.contiguous(), scale.contiguous(), bias.contiguous()


def random_q4(N, K, device, *seed_parts, std=0.02, chunk_rows=16384):
    """A seeded N(0, std) matrix [N][K], quantised; generated in row chunks to bound memory."""
    g = _gen(device, *seed_parts)
    qs, ss, bs = [], [], []
    for r0 in range(0, N, chunk_rows):
        rows = min(chunk_rows, N - r0)
        w = torch.randn(rows, K, generator=g, device=device, dtype=torch.float32) * std
        q, s, b = quantize_q4(w)
        qs.append(q), ss.append(s), bs.append(b)
    return torch.cat(qs), torch.cat(ss), torch.cat(bs)


def norm_weight(n, device, *seed_parts):
    g = _gen(device, *seed_parts)
    return (1.0 + 0.02 * torch.randn(n, generator=g, device=device, dtype=torch.float32)).to(torch.bfloat16)


def rope_table(max_positions, head_dim, base, device="cpu"):
    """float32 [max_positions][head_dim/2][2] = (cos, sin) of position * base^(-2i/head_dim), from fp64."""
    half = head_dim // 2
    inv = np.power(float(base), -np.arange(half, dtype=np.float64) * 2.0 / head_dim)
    ang = np.arange(max_positions, dtype=np.float64)[:, None] * inv[None, :]
    tab = np.stack([np.cos(ang), np.sin(ang)], axis=-1).astype(np.float32)
    return torch.from_numpy(tab).to(device)


# -------------------------------------------------------------------- weights

def make_weights(shape, seed=0, device="cpu"):
    """All arrays of a model as a nested dict (see oracle.q4d_oracle.OracleModel for the keys)."""
    H, d = shape.hidden, shape.head_dim
    layers = []
    for l in range(shape.n_layers):
        lw = {
            "attn_norm": norm_weight(H, device, seed, shape.name, l, "attn_norm"),
            "mlp_norm": norm_weight(H, device, seed, shape.name, l, "mlp_norm"),
            "q_norm": norm_weight(d, device, seed, shape.name, l, "q_norm") if shape.qk_norm else None,
            "k_norm": norm_weight(d, device, seed, shape.name, l, "k_norm") if shape.qk_norm else None,
            "wqkv": random_q4(shape.qkv_out, H, device, seed, shape.name, l, "wqkv"),
            "wo": random_q4(H, shape.n_q_heads * d, device, seed, shape.name, l, "wo"),
        }
        if shape.n_experts:
            E, Ie = shape.n_experts, shape.expert_inter
            g = _gen(device, seed, shape.name, l, "router")
            lw["router"] = (0.02 * torch.randn(E, H, generator=g, device=device, dtype=torch.float32)).to(torch.bfloat16)
            lw["experts_gate_up"] = random_q4(E * 2 * Ie, H, device, seed, shape.name, l, "experts_gate_up")
            lw["experts_down"] = random_q4(E * H, Ie, device, seed, shape.name, l, "experts_down")
        else:
            lw["w_gate_up"] = random_q4(2 * shape.mlp_inter, H, device, seed, shape.name, l, "w_gate_up")
            lw["w_down"] = random_q4(H, shape.mlp_inter, device, seed, shape.name, l, "w_down")
        layers.append(lw)
    embed = random_q4(shape.vocab, H, device, seed, shape.name, "embed")
    lm_head = embed if shape.tie_embeddings else random_q4(shape.vocab, H, device, seed, shape.name, "lm_head")
    return {
        "layers": layers,
        "final_norm": norm_weight(H, device, seed, shape.name, "final_norm"),
        "embed": embed,
        "lm_head": lm_head,
        "rope": rope_table(shape.max_positions, d, shape.rope_base, device),
    }


# -------------------------------------------------------------------- KV pool

def pool_shape(shape, num_blocks, block_size=BLOCK_SIZE):
    return (shape.n_layers, 2, num_blocks, shape.n_kv_heads, block_size, shape.head_dim)


def make_pool(shape, num_blocks, device="cpu", block_size=BLOCK_SIZE):
    return torch.zeros(pool_shape(shape, num_blocks, block_size), dtype=torch.bfloat16, device=device)


class BlockAllocator:
    """Free list of physical block ids, shuffled so block tables are non-contiguous."""

    def __init__(self, num_blocks, seed=0):
        rng = np.random.default_rng(_seed(seed, "blocks") % (2 ** 32))
        self.free = list(rng.permutation(num_blocks).astype(int))

    def alloc(self, k):
        if k > len(self.free):
            raise RuntimeError("KV pool exhausted")
        out, self.free = self.free[:k], self.free[k:]
        return out

    def release(self, ids):
        self.free.extend(int(i) for i in ids)


def fill_blocks(pool, block_ids, *seed_parts, layers_per_chunk=4):
    """Overwrite whole blocks (all layers, K and V, every slot) with seeded N(0, 1) bf16 values."""
    L, _, _, nkv, bs, d = pool.shape
    idx = torch.as_tensor(list(block_ids), dtype=torch.long, device=pool.device)
    if idx.numel() == 0:
        return
    g = _gen(pool.device, *seed_parts)
    for l0 in range(0, L, layers_per_chunk):
        ls = min(layers_per_chunk, L - l0)
        vals = torch.randn(ls, 2, idx.numel(), nkv, bs, d, generator=g, device=pool.device,
                           dtype=torch.float32).to(torch.bfloat16)
        pool[l0:l0 + ls].index_copy_(2, idx, vals)


# ------------------------------------------------------------ request lengths

def draw_lengths(n, lo, hi, rng, log_uniform=False):
    if log_uniform:
        return np.exp(rng.uniform(math.log(lo), math.log(hi), size=n)).astype(np.int64).clip(lo, hi)
    return rng.integers(lo, hi + 1, size=n).astype(np.int64)


class Request:
    __slots__ = ("rid", "length", "blocks", "token")

    def __init__(self, rid, length, blocks, token):
        self.rid, self.length, self.blocks, self.token = rid, length, blocks, token


class ChurnScript:
    """The admit/release schedule of the continuous-batching loop, scripted.

    n requests start with prefilled lengths drawn from [lo, hi]; every
    `churn_every` steps `churn_count` random active requests finish and as many
    new ones are admitted with `admit_len` prefilled tokens.  The object owns the
    block allocator and the per-request block lists; `step_inputs()` returns the
    arrays one decode step takes and `advance()` records that each active request
    grew by one token.
    """

    def __init__(self, shape, pool, n, lo, hi, log_uniform=False, churn_every=32, churn_count=4,
                 admit_len=512, seed=0, block_size=BLOCK_SIZE):
        self.shape, self.pool, self.bs, self.seed = shape, pool, block_size, seed
        self.rng = np.random.default_rng(_seed(seed, "script") % (2 ** 32))
        self.alloc = BlockAllocator(pool.shape[2], seed)
        self.churn_every, self.churn_count, self.admit_len = churn_every, churn_count, admit_len
        self.next_rid = 0
        self.step = 0
        self.active = []
        self.pending = []  # the queue Q of Algorithm 1: requests whose prefilled KV is already in the pool
        self.events = []  # ("admit", rid, len) / ("release", rid) since the last step
        for length in draw_lengths(n, lo, hi, self.rng, log_uniform):
            self._admit(int(length))

    def _make_request(self, length):
        rid = self.next_rid
        self.next_rid += 1
        nblk = (length + 1 + self.bs - 1) // self.bs
        blocks = self.alloc.alloc(nblk)
        fill_blocks(self.pool, blocks, self.seed, "kv", rid)
        tok = int(self.rng.integers(0, self.shape.vocab))
        return Request(rid, length, blocks, tok)

    def _admit(self, length):
        r = self.pending.pop(0) if self.pending else self._make_request(length)
        self.active.append(r)
        self.events.append(("admit", r.rid, r.length))

    def prepare_pending(self, steps):
        """Create ahead of time the requests that will be admitted during the next `steps` steps, so that
        admitting them later is bookkeeping only (their prefilled KV is written now)."""
        if not self.churn_every:
            return
        due = sum(1 for s in range(self.step + 1, self.step + steps + 1) if s % self.churn_every == 0)
        while len(self.pending) < due * self.churn_count:
            self.pending.append(self._make_request(self.admit_len))

    def churn(self):
        """Apply the between-steps membership change due before the coming step, if any."""
        if self.step > 0 and self.churn_every and self.step % self.churn_every == 0:
            k = min(self.churn_count, len(self.active))
            out = sorted(self.rng.choice(len(self.active), size=k, replace=False).tolist(), reverse=True)
            for i in out:
                r = self.active.pop(i)
                self.alloc.release(r.blocks)
                self.events.append(("release", r.rid))
            for _ in range(k):
                self._admit(self.admit_len)

    def pop_events(self):
        ev, self.events = self.events, []
        return ev

    def step_inputs(self):
        """(request ids int64 [n], last tokens int32 [n], lens int32 [n], block tables int32 [n][max_blocks])."""
        for r in self.active:  # the new token needs a slot
            need = (r.length + 1 + self.bs - 1) // self.bs
            if need > len(r.blocks):
                r.blocks.extend(self.alloc.alloc(need - len(r.blocks)))
        mb = max(len(r.blocks) for r in self.active)
        bt = np.zeros((len(self.active), mb), dtype=np.int32)
        for i, r in enumerate(self.active):
            bt[i, :len(r.blocks)] = r.blocks
        ids = np.array([r.rid for r in self.active], dtype=np.int64)
        toks = np.array([r.token for r in self.active], dtype=np.int32)
        lens = np.array([r.length for r in self.active], dtype=np.int32)
        return ids, toks, lens, bt

    def advance(self, next_tokens=None):
        for i, r in enumerate(self.active):
            r.length += 1
            if next_tokens is not None:
                r.token = int(next_tokens[i])
        self.step += 1

    def kv_tokens_read(self):
        """Tokens whose K and V the coming step reads (new token included)."""
        return int(sum(r.length + 1 for r in self.active))
