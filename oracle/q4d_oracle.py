"""ctypes binding of the CPU oracle (oracle/q4d_oracle.c).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU
baseline use it; the CUDA library never does and shares nothing with it.

Arrays are numpy: packed codes uint32, bf16 as uint16 bit patterns, tables and
logits float32.  Torch tensors are accepted where noted and converted by bit
pattern (bfloat16 -> uint16, int32 -> uint32).
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

_LIB = None


class Shape(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("n_layers", "hidden", "n_q_heads", "n_kv_heads", "head_dim",
                                          "mlp_inter", "vocab", "group_size", "bits", "qk_norm",
                                          "tie_embeddings")] + [("rms_eps", C.c_float)] + \
               [(k, C.c_int32) for k in ("n_experts", "top_k", "expert_inter", "norm_topk_prob",
                                          "max_batch", "max_positions")]


class QTensor(C.Structure):
    _fields_ = [("q", C.c_void_p), ("scales", C.c_void_p), ("biases", C.c_void_p)]


class Layer(C.Structure):
    _fields_ = [("attn_norm", C.c_void_p), ("mlp_norm", C.c_void_p), ("q_norm", C.c_void_p),
                ("k_norm", C.c_void_p), ("wqkv", QTensor), ("wo", QTensor), ("w_gate_up", QTensor),
                ("w_down", QTensor), ("router", C.c_void_p), ("experts_gate_up", QTensor),
                ("experts_down", QTensor)]


class Weights(C.Structure):
    _fields_ = [("layers", C.POINTER(Layer)), ("final_norm", C.c_void_p), ("embed", QTensor),
                ("lm_head", QTensor), ("rope_cos_sin", C.c_void_p)]


def _declare(L):
    L.orc_bf16_round.restype = C.c_uint16
    L.orc_bf16_round.argtypes = [C.c_double]
    L.orc_bf16_to_float.restype = C.c_float
    L.orc_bf16_to_float.argtypes = [C.c_uint16]
    L.orc_num_threads.restype = C.c_int
    for name in ("orc_q4_matmul", "orc_attention_head", "orc_attention_paged", "orc_decode_step"):
        getattr(L, name).restype = C.c_int
    return L


def lib():
    global _LIB
    if _LIB is None:
        _LIB = _declare(C.CDLL(_build.build()))
    return _LIB


def to_np(t, dtype=None):
    """numpy view of a numpy array or a CPU copy of a torch tensor, by bit pattern."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        a = t
    else:
        import torch
        t = t.detach().cpu().contiguous()
        if t.dtype == torch.bfloat16:
            a = t.view(torch.int16).numpy().view(np.uint16)
        elif t.dtype == torch.int32:
            a = t.numpy()
        else:
            a = t.numpy()
    if dtype is not None and a.dtype != dtype:
        if a.dtype.itemsize == np.dtype(dtype).itemsize and a.dtype.kind in "iu" and np.dtype(dtype).kind in "iu":
            a = a.view(dtype)
        else:
            a = a.astype(dtype)
    return np.ascontiguousarray(a)


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


# ----------------------------------------------------------------- elementary ops

def bf16_round(values):
    """fp64 array -> bf16 bit patterns (uint16), round to nearest even, one rounding."""
    v = np.ascontiguousarray(values, dtype=np.float64)
    out = np.empty(v.shape, dtype=np.uint16)
    lib().orc_bf16_round_array(_p(v), C.c_int64(v.size), _p(out))
    return out


def bf16_to_f64(bits):
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def quantize_q4(w):
    w = np.ascontiguousarray(w, dtype=np.float32)
    N, K = w.shape
    assert K % 64 == 0
    q = np.empty((N, K // 8), dtype=np.uint32)
    s = np.empty((N, K // 64), dtype=np.uint16)
    b = np.empty((N, K // 64), dtype=np.uint16)
    lib().orc_quantize_q4(_p(w), C.c_int64(N), C.c_int64(K), _p(q), _p(s), _p(b))
    return q, s, b


def dequant_q4(q, s, b):
    q, s, b = to_np(q, np.uint32), to_np(s, np.uint16), to_np(b, np.uint16)
    N, K = q.shape[0], q.shape[1] * 8
    out = np.empty((N, K), dtype=np.float32)
    lib().orc_dequant_q4(_p(q), _p(s), _p(b), C.c_int64(N), C.c_int64(K), _p(out))
    return out


def q4_matmul(q, s, b, x_bits):
    """x bf16 bits [n][K] -> fp64 [n][N], unrounded."""
    q, s, b = to_np(q, np.uint32), to_np(s, np.uint16), to_np(b, np.uint16)
    x = to_np(x_bits, np.uint16)
    N, K = q.shape[0], q.shape[1] * 8
    n = x.shape[0]
    assert x.shape[1] == K
    out = np.empty((n, N), dtype=np.float64)
    rc = lib().orc_q4_matmul(_p(q), _p(s), _p(b), C.c_int64(N), C.c_int64(K), _p(x), C.c_int32(n), _p(out))
    assert rc == 0, rc
    return out


def rmsnorm(x_bits, w_bits, eps):
    x, w = to_np(x_bits, np.uint16), to_np(w_bits, np.uint16)
    n, H = x.shape
    y = np.empty_like(x)
    lib().orc_rmsnorm(_p(x), _p(w), C.c_float(eps), C.c_int32(n), C.c_int32(H), _p(y))
    return y


def rope(head_bits, cs_row):
    """One head (bf16 bits [d]) rotated with the table row cs_row float32 [d/2][2]."""
    h = to_np(head_bits, np.uint16).copy()
    cs = np.ascontiguousarray(cs_row, dtype=np.float32)
    lib().orc_rope(_p(h), _p(cs), C.c_int32(h.size))
    return h


def silu_mul(g_bits, u_bits):
    g, u = to_np(g_bits, np.uint16), to_np(u_bits, np.uint16)
    h = np.empty_like(g)
    lib().orc_silu_mul(_p(g), _p(u), C.c_int64(g.size), _p(h))
    return h


def argmax(logits):
    lg = np.ascontiguousarray(logits, dtype=np.float32)
    n, V = lg.shape
    out = np.empty(n, dtype=np.int32)
    lib().orc_argmax(_p(lg), C.c_int32(n), C.c_int64(V), _p(out))
    return out


def moe_route(z, top_k, norm):
    z = np.ascontiguousarray(z, dtype=np.float64)
    idx = np.empty(top_k, dtype=np.int32)
    wgt = np.empty(top_k, dtype=np.float64)
    lib().orc_moe_route(_p(z), C.c_int32(z.size), C.c_int32(top_k), C.c_int32(int(norm)), _p(idx), _p(wgt))
    return idx, wgt


def attention_head(q_bits, K_bits, V_bits):
    q, K, V = to_np(q_bits, np.uint16), to_np(K_bits, np.uint16), to_np(V_bits, np.uint16)
    T, d = K.shape
    out = np.empty(d, dtype=np.uint16)
    rc = lib().orc_attention_head(_p(q), _p(K), _p(V), C.c_int32(T), C.c_int32(d), _p(out))
    assert rc == 0, rc
    return out


def kv_gather(pool, nkv, bs, d, layer, head, block_table, length):
    """pool uint16 [L][2][blocks][nkv][bs][d] -> contiguous K, V [length][d]."""
    pool = to_np(pool, np.uint16)
    bt = np.ascontiguousarray(block_table, dtype=np.int32)
    num_blocks = pool.shape[2]
    k = np.empty((length, d), dtype=np.uint16)
    v = np.empty((length, d), dtype=np.uint16)
    lib().orc_kv_gather(_p(pool), C.c_int32(num_blocks), C.c_int32(nkv), C.c_int32(bs), C.c_int32(d),
                        C.c_int32(layer), C.c_int32(head), _p(bt), C.c_int32(length), _p(k), _p(v))
    return k, v


def attention_paged(q_bits, pool, nq, nkv, bs, d, layer, lens, block_tables):
    q = to_np(q_bits, np.uint16)
    pool = to_np(pool, np.uint16)
    lens = np.ascontiguousarray(lens, dtype=np.int32)
    bt = np.ascontiguousarray(block_tables, dtype=np.int32)
    n = lens.size
    out = np.empty((n, nq, d), dtype=np.uint16)
    rc = lib().orc_attention_paged(_p(q), _p(pool), C.c_int32(pool.shape[2]), C.c_int32(nq), C.c_int32(nkv),
                                   C.c_int32(bs), C.c_int32(d), C.c_int32(layer), C.c_int32(n), _p(lens),
                                   _p(bt), C.c_int32(bt.shape[1]), _p(out))
    assert rc == 0, rc
    return out


def num_threads():
    return int(lib().orc_num_threads())


# ----------------------------------------------------------------- whole model

_SHAPE_KEYS = [f[0] for f in Shape._fields_]


class OracleModel:
    """Host copy of a model's arrays laid out for orc_decode_step.

    `shape` is any object with the attributes of the Shape struct; `weights` is
    the nested dict produced by the workload generator (torch tensors or numpy
    arrays): per layer attn_norm, mlp_norm, q_norm, k_norm, wqkv, wo, w_gate_up,
    w_down (each a (q, scales, biases) triple), router, experts_gate_up,
    experts_down; plus final_norm, embed, lm_head, rope.
    """

    def __init__(self, shape, weights):
        self.shape = Shape(**{k: (float(getattr(shape, k)) if k == "rms_eps" else int(getattr(shape, k)))
                              for k in _SHAPE_KEYS})
        self._keep = []
        n_layers = self.shape.n_layers
        self._layers = (Layer * n_layers)()
        for i, lw in enumerate(weights["layers"]):
            L = self._layers[i]
            for k in ("attn_norm", "mlp_norm", "q_norm", "k_norm", "router"):
                setattr(L, k, self._ptr(lw.get(k), np.uint16))
            for k in ("wqkv", "wo", "w_gate_up", "w_down", "experts_gate_up", "experts_down"):
                setattr(L, k, self._qt(lw.get(k)))
        self.weights = Weights()
        self.weights.layers = C.cast(self._layers, C.POINTER(Layer))
        self.weights.final_norm = self._ptr(weights["final_norm"], np.uint16)
        self.weights.embed = self._qt(weights["embed"])
        self.weights.lm_head = self._qt(weights["lm_head"])
        self.weights.rope_cos_sin = self._ptr(weights["rope"], np.float32)

    def _ptr(self, t, dtype):
        if t is None:
            return None
        a = to_np(t, dtype)
        self._keep.append(a)
        return a.ctypes.data

    def _qt(self, triple):
        qt = QTensor()
        if triple is not None:
            qt.q = self._ptr(triple[0], np.uint32)
            qt.scales = self._ptr(triple[1], np.uint16)
            qt.biases = self._ptr(triple[2], np.uint16)
        return qt

    def decode_step(self, pool, block_size, lens, last_tokens, block_tables, layer_limit=-1,
                    want_logits=True, want_taps=False):
        """pool: numpy uint16 [L][2][blocks][nkv][bs][d], updated in place.
        Returns (next_tokens int32 [n], logits float32 [n][V] or None, taps or None)."""
        assert isinstance(pool, np.ndarray) and pool.dtype == np.uint16 and pool.flags.c_contiguous
        lens = np.ascontiguousarray(lens, dtype=np.int32)
        toks = np.ascontiguousarray(last_tokens, dtype=np.int32)
        bt = np.ascontiguousarray(block_tables, dtype=np.int32)
        n = lens.size
        sh = self.shape
        nxt = np.empty(n, dtype=np.int32)
        logits = np.empty((n, sh.vocab), dtype=np.float32) if want_logits else None
        taps = np.zeros((sh.n_layers + 1, n, sh.hidden), dtype=np.uint16) if want_taps else None
        rc = lib().orc_decode_step(C.byref(sh), C.byref(self.weights), _p(pool), C.c_int32(pool.shape[2]),
                                   C.c_int32(block_size), C.c_int32(n), _p(lens), _p(toks), _p(bt),
                                   C.c_int32(bt.shape[1] if n else 0), C.c_int32(layer_limit), _p(nxt),
                                   _p(logits), _p(taps))
        if rc != 0:
            raise RuntimeError(f"orc_decode_step failed: {rc}")
        return nxt, logits, taps


# ------------------------------------------------------------------ prompt processing
def prefill(model, pool, block_size, tokens, start_pos, block_table):
    """Prompt processing for one request (Section 3.2: the forward pass over the prompt tokens that a prefix-cache
    hit skips up to start_pos).  By definition it is the decode step applied to the prompt's tokens one after the
    other, each at its position, over the same pool: K, V of tokens[start_pos:] are appended in place, and the result
    of the last step (greedy token after the prompt, its logits) is returned."""
    bt = np.ascontiguousarray(block_table, dtype=np.int32).reshape(1, -1)
    nxt = logits = None
    for pos in range(int(start_pos), len(tokens)):
        nxt, logits, _ = model.decode_step(pool, block_size, [pos], [int(tokens[pos])], bt)
    return int(nxt[0]), logits[0]


# ------------------------------------------------------------------ sampling
# The paper's scheduler generates "a token" per request (Algorithm 1, generation loop) and says nothing about how
# it is chosen.  The reading built here is the usual temperature / top-k / top-p rule with the random draw u given by
# the caller, written out plainly (a sort, a running sum) in fp64 with integer weights:
#   w_j = rint(2^40 exp((l_j - max l) / T));  top-k keeps logits >= the k-th largest (ties at the cut stay);
#   top-p keeps logits >= c for the largest c whose set weighs >= ceil(top_p * kept weight);
#   t = floor(u * W) over the kept weight W; walk by (descending logit, ascending index); first running weight > t.

def sampling_table(logits, temperature, top_k, top_p):
    """(order, weights in that order, number of kept tokens): `order` lists all token ids by descending logit and
    ascending index among equal logits; the first `kept` of them survive top-k and top-p."""
    l = np.asarray(logits, dtype=np.float64)
    V = l.size
    order = np.lexsort((np.arange(V), -l))
    ls = l[order]
    w = np.rint(np.exp((ls - ls[0]) / float(temperature)) * 2.0 ** 40).astype(np.int64)
    kept = V
    if 0 < top_k < V:
        kth = ls[top_k - 1]
        kept = int(np.searchsorted(-ls, -kth, side="right"))          # every logit >= the k-th largest
    if top_p < 1.0:
        Wk = int(w[:kept].sum())
        target = min(max(int(np.ceil(float(np.float32(top_p)) * float(Wk))), 1), Wk)
        cum = np.cumsum(w[:kept])
        first = int(np.searchsorted(cum, target, side="left"))         # first position whose running weight >= target
        c = ls[first]
        kept = min(kept, int(np.searchsorted(-ls, -c, side="right")))  # and every token tied with it
    return order, w, kept


def sample_token(logits, temperature, top_k, top_p, u):
    """The token the rule draws for one request."""
    l = np.asarray(logits, dtype=np.float64)
    if not temperature > 0.0:
        return int(np.flatnonzero(l == l.max())[0])
    order, w, kept = sampling_table(l, temperature, top_k, top_p)
    W = int(w[:kept].sum())
    t = min(int(float(np.float32(u)) * float(W)), W - 1)
    cum = np.cumsum(w[:kept])
    return int(order[int(np.searchsorted(cum, t, side="right"))])      # first running weight > t
