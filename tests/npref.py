"""Independent numpy restatement used to pin the C oracle (never used by the product).

Written separately from oracle/q4d_oracle.c: bf16 rounding by integer bit
manipulation of the fp64 pattern, weights as explicit float matrices, library
matmul, full-matrix softmax, contiguous KV.  Toy sizes only.
"""
import numpy as np


def bf16_bits(v):
    """fp64 -> bf16 bit patterns, ties to even, by integer arithmetic (normal range and zero only)."""
    v = np.ascontiguousarray(v, dtype=np.float64)
    bits = v.view(np.uint64)
    drop = np.uint64(45)  # 52 fraction bits -> 7
    lsb = (bits >> drop) & np.uint64(1)
    rounded = (bits + lsb + np.uint64((1 << 44) - 1)) >> drop  # sign(1) exp(11) frac(7)
    sign = (rounded >> np.uint64(18)) & np.uint64(1)
    e11 = ((rounded >> np.uint64(7)) & np.uint64(0x7FF)).astype(np.int64)
    frac = rounded & np.uint64(0x7F)
    zero = (v == 0)
    e8 = e11 - 1023 + 127
    assert np.all(zero | ((e8 >= 1) & (e8 <= 254))), "outside the bf16 normal range"
    out = (sign << np.uint64(15)) | (e8.astype(np.uint64) << np.uint64(7)) | frac
    out = np.where(zero, sign << np.uint64(15), out)
    return out.astype(np.uint16)


def bf16_val(bits):
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def rbf(v):
    """Round fp64 values to bf16 and return them as fp64."""
    return bf16_val(bf16_bits(v))


def unpack_codes(q):
    """uint32 [N][K/8] -> integer codes [N][K]: element k in word k>>3, bits 4*(k&7).."""
    q = np.asarray(q).view(np.uint32)
    N, W = q.shape
    out = np.zeros((N, W * 8), dtype=np.int64)
    for i in range(8):
        out[:, i::8] = (q >> np.uint32(4 * i)) & np.uint32(0xF)
    return out


def dense_matrix(triple):
    """(codes, scales bf16 bits, biases bf16 bits) -> float64 matrix of fp32-rounded weights."""
    q, s, b = triple
    codes = unpack_codes(q).astype(np.float64)
    s64 = np.repeat(bf16_val(s), 64, axis=1)
    b64 = np.repeat(bf16_val(b), 64, axis=1)
    return (s64 * codes + b64).astype(np.float32).astype(np.float64)  # s*q+b is exact in fp64 here


def rmsnorm(x, w, eps):
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return rbf(x / np.sqrt(ms + np.float64(np.float32(eps))) * w)


def rope(h, cs):
    """h [..., d] fp64, cs [d/2][2] float32."""
    d = h.shape[-1]
    a, b = h[..., : d // 2], h[..., d // 2:]
    c, s = cs[:, 0].astype(np.float64), cs[:, 1].astype(np.float64)
    return rbf(np.concatenate([a * c - b * s, b * c + a * s], axis=-1))


def softmax(z):
    e = np.exp(z - np.max(z, axis=-1, keepdims=True))
    return e / np.sum(e, axis=-1, keepdims=True)


def attention(q, K, V):
    """q [G][d], K, V [T][d] fp64 -> bf16-rounded [G][d] via the full score matrix."""
    S = q @ K.T / np.sqrt(q.shape[-1])
    return rbf(softmax(S) @ V)


def silu(g):
    return g / (1.0 + np.exp(-g))


def decode_step(shape, W, kv, lens, tokens):
    """Whole decode step on contiguous per-request KV.

    W: dict of float64 matrices / vectors (see tests/test_oracle_step.py); kv[r][l] = (K [len][nkv][d],
    V [len][nkv][d]) fp64.  Returns (next tokens, logits float32 [n][V], new (k, v) per request and layer,
    hidden taps [L+1][n][H]).
    """
    H, d, nq, nkv = shape.hidden, shape.head_dim, shape.n_q_heads, shape.n_kv_heads
    G = nq // nkv
    out_logits, new_kv, taps = [], [], []
    for r, tok in enumerate(tokens):
        x = rbf(W["embed"][tok])
        tap = [x.copy()]
        nk = []
        for l in range(shape.n_layers):
            lw = W["layers"][l]
            y = rmsnorm(x, lw["attn_norm"], shape.rms_eps)
            qkv = rbf(lw["wqkv"] @ y).reshape(nq + 2 * nkv, d)
            qh, kh, vh = qkv[:nq], qkv[nq:nq + nkv], qkv[nq + nkv:]
            if shape.qk_norm:
                qh = rmsnorm(qh, lw["q_norm"], shape.rms_eps)
                kh = rmsnorm(kh, lw["k_norm"], shape.rms_eps)
            cs = W["rope"][lens[r]]
            qh, kh = rope(qh, cs), rope(kh, cs)
            Kc = np.concatenate([kv[r][l][0], kh[None]], axis=0)
            Vc = np.concatenate([kv[r][l][1], vh[None]], axis=0)
            nk.append((kh, vh))
            att = np.concatenate([attention(qh[h * G:(h + 1) * G], Kc[:, h], Vc[:, h]) for h in range(nkv)])
            x = rbf(x + rbf(lw["wo"] @ att.reshape(-1)))
            y = rmsnorm(x, lw["mlp_norm"], shape.rms_eps)
            if shape.n_experts:
                z = lw["router"] @ y
                p = softmax(z)
                order = sorted(range(shape.n_experts), key=lambda e: (-z[e], e))[: shape.top_k]
                pw = p[order] / (p[order].sum() if shape.norm_topk_prob else 1.0)
                mix = np.zeros(H)
                for e, pe in zip(order, pw):
                    gu = rbf(lw["experts_gate_up"][e] @ y)
                    Ie = shape.expert_inter
                    h_ = rbf(silu(gu[:Ie]) * gu[Ie:])
                    mix += pe * rbf(lw["experts_down"][e] @ h_)
                x = rbf(x + rbf(mix))
            else:
                gu = rbf(lw["w_gate_up"] @ y)
                I = shape.mlp_inter
                h_ = rbf(silu(gu[:I]) * gu[I:])
                x = rbf(x + rbf(lw["w_down"] @ h_))
            tap.append(x.copy())
        y = rmsnorm(x, W["final_norm"], shape.rms_eps)
        out_logits.append((W["lm_head"] @ y).astype(np.float32))
        new_kv.append(nk)
        taps.append(tap)
    logits = np.stack(out_logits)
    nxt = np.array([int(np.flatnonzero(row == row.max())[0]) for row in logits], dtype=np.int32)
    taps = np.stack([np.stack(t) for t in taps], axis=1)  # [L+1][n][H]
    return nxt, logits, new_kv, taps
