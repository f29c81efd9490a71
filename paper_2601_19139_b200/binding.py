"""ctypes binding of libq4decode.so: argument marshalling only.

Every function here forwards to the C entry point of the same name
(include/q4decode.h); all computation happens in the CUDA library.  There is
no fallback: if the shared library is missing or a call fails, an exception is
raised.  PyTorch is used for device memory and streams only.
"""
import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libq4decode.so")

K_NAMES = ["embed", "rmsnorm", "gemm_qkv", "rope_append", "attention", "attn_merge", "gemm_o", "gemm_gate_up",
           "gemm_down", "moe_router", "moe_gate_up", "moe_down", "lm_head", "argmax", "fused_step"]

EXPORTS = [
    "q4d_last_error", "q4d_model_workspace_bytes", "q4d_model_create", "q4d_model_destroy", "q4d_kv_pool_bytes",
    "q4d_kv_pool_create", "q4d_kv_pool_destroy", "q4d_request_admit", "q4d_request_release", "q4d_request_len",
    "q4d_request_count", "q4d_decode_step", "q4d_decode_step_chained", "q4d_decode_step_host", "q4d_decode_step_sampled", "q4d_sample", "q4d_prefill", "q4d_profile_enable",
    "q4d_profile_read", "q4d_launch_count", "q4d_step_is_fused", "q4d_timeline_enable", "q4d_timeline_read",
    "q4d_step_io_bytes", "q4d_moe_touched_experts", "q4d_op_scratch_bytes", "q4d_q4_gemm",
    "q4d_q4_gemm_noalloc", "q4d_noalloc_max_scratch_bytes",
    "q4d_rmsnorm", "q4d_embed", "q4d_rope_append", "q4d_paged_attention", "q4d_argmax", "q4d_debug_dequant",
    "q4d_debug_kv_gather", "q4d_debug_run_layers", "q4d_debug_set_status",
    "q4d_sha256", "q4d_prefix_cache_create", "q4d_prefix_cache_destroy", "q4d_prefix_lookup", "q4d_prefix_insert",
    "q4d_prefix_release", "q4d_prefix_evict", "q4d_prefix_cache_stats", "q4d_content_cache_create",
    "q4d_content_cache_destroy", "q4d_content_lookup", "q4d_content_store", "q4d_content_release", "q4d_content_evict",
    "q4d_content_cache_stats",
]


class Q4dError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"q4decode error {code}: {msg}")
        self.code = code


class ShapeStruct(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("n_layers", "hidden", "n_q_heads", "n_kv_heads", "head_dim", "mlp_inter",
                                          "vocab", "group_size", "bits", "qk_norm", "tie_embeddings")] + \
               [("rms_eps", C.c_float)] + \
               [(k, C.c_int32) for k in ("n_experts", "top_k", "expert_inter", "norm_topk_prob", "max_batch",
                                          "max_positions")]


class QTensor(C.Structure):
    _fields_ = [("q", C.c_void_p), ("scales", C.c_void_p), ("biases", C.c_void_p)]


class LayerWeights(C.Structure):
    _fields_ = [("attn_norm", C.c_void_p), ("mlp_norm", C.c_void_p), ("q_norm", C.c_void_p), ("k_norm", C.c_void_p),
                ("wqkv", QTensor), ("wo", QTensor), ("w_gate_up", QTensor), ("w_down", QTensor),
                ("router", C.c_void_p), ("experts_gate_up", QTensor), ("experts_down", QTensor)]


class WeightsStruct(C.Structure):
    _fields_ = [("layers", C.POINTER(LayerWeights)), ("final_norm", C.c_void_p), ("embed", QTensor),
                ("lm_head", QTensor), ("rope_cos_sin", C.c_void_p)]


_LIB = None


def lib():
    """The loaded shared library; raises if it has not been built."""
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2601_19139_b200.build` (needs nvcc)")
        L = C.CDLL(LIB_PATH)
        L.q4d_last_error.restype = C.c_char_p
        L.q4d_model_workspace_bytes.restype = C.c_size_t
        L.q4d_kv_pool_bytes.restype = C.c_size_t
        L.q4d_op_scratch_bytes.restype = C.c_size_t
        L.q4d_launch_count.restype = C.c_int64
        L.q4d_noalloc_max_scratch_bytes.restype = C.c_size_t
        _LIB = L
    return _LIB


def _check(rc):
    if rc != 0:
        raise Q4dError(rc, lib().q4d_last_error().decode())


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        assert t.is_contiguous()
        return C.c_void_p(t.data_ptr())
    if isinstance(t, np.ndarray):
        assert t.flags.c_contiguous
        return C.c_void_p(t.ctypes.data)
    return C.c_void_p(int(t))


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _qt(triple):
    qt = QTensor()
    if triple is not None:
        qt.q, qt.scales, qt.biases = (t.data_ptr() for t in triple)
    return qt


def shape_struct(shape):
    return ShapeStruct(**{k: (float(getattr(shape, k)) if k == "rms_eps" else int(getattr(shape, k)))
                          for k, _ in ShapeStruct._fields_})


# ------------------------------------------------------------------ objects

class Model:
    """q4d_model_create / q4d_model_destroy around a dict of device tensors (workload.gen.make_weights)."""

    def __init__(self, shape, weights, device="cuda"):
        L = lib()
        self.shape = shape
        self.sh = shape_struct(shape)
        self.weights = weights  # keeps the tensors alive
        self._layers = (LayerWeights * shape.n_layers)()
        for i, lw in enumerate(weights["layers"]):
            S = self._layers[i]
            for k in ("attn_norm", "mlp_norm", "q_norm", "k_norm", "router"):
                t = lw.get(k)
                setattr(S, k, None if t is None else t.data_ptr())
            for k in ("wqkv", "wo", "w_gate_up", "w_down", "experts_gate_up", "experts_down"):
                setattr(S, k, _qt(lw.get(k)))
        self._w = WeightsStruct()
        self._w.layers = C.cast(self._layers, C.POINTER(LayerWeights))
        self._w.final_norm = weights["final_norm"].data_ptr()
        self._w.embed = _qt(weights["embed"])
        self._w.lm_head = _qt(weights["lm_head"])
        self._w.rope_cos_sin = weights["rope"].data_ptr()
        nbytes = L.q4d_model_workspace_bytes(C.byref(self.sh))
        if nbytes == 0:
            raise Q4dError(-11, L.q4d_last_error().decode())
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=device)
        self.handle = C.c_void_p()
        _check(L.q4d_model_create(C.byref(self.sh), C.byref(self._w), _ptr(self.workspace), C.c_size_t(nbytes),
                                  C.byref(self.handle)))

    def close(self):
        if self.handle:
            lib().q4d_model_destroy(self.handle)
            self.handle = C.c_void_p()

    def profile_enable(self, on=True):
        _check(lib().q4d_profile_enable(self.handle, C.c_int32(int(on))))

    def profile_read(self):
        ms = (C.c_float * len(K_NAMES))()
        cnt = (C.c_int32 * len(K_NAMES))()
        _check(lib().q4d_profile_read(self.handle, ms, cnt))
        return {k: (float(ms[i]), int(cnt[i])) for i, k in enumerate(K_NAMES)}

    def launch_count(self):
        return int(lib().q4d_launch_count(self.handle))

    def is_fused(self):
        return bool(lib().q4d_step_is_fused(self.handle))

    def timeline_enable(self, on=True):
        _check(lib().q4d_timeline_enable(self.handle, int(on)))

    def timeline_read(self):
        us = (C.c_float * len(K_NAMES))()
        cnt = (C.c_int32 * len(K_NAMES))()
        _check(lib().q4d_timeline_read(self.handle, us, cnt))
        return {k: (float(us[i]), int(cnt[i])) for i, k in enumerate(K_NAMES) if cnt[i]}

    def step_io_bytes(self):
        h2d, d2h = C.c_int64(), C.c_int64()
        _check(lib().q4d_step_io_bytes(self.handle, C.byref(h2d), C.byref(d2h)))
        return h2d.value, d2h.value

    def debug_set_status(self, value):
        _check(lib().q4d_debug_set_status(self.handle, C.c_uint32(value)))

    def moe_touched_experts(self):
        total = C.c_int64()
        _check(lib().q4d_moe_touched_experts(self.handle, C.byref(total)))
        return total.value


class KVPool:
    """q4d_kv_pool_create over a torch bf16 tensor [L][2][blocks][nkv][16][128]."""

    def __init__(self, model, pool_tensor):
        L = lib()
        self.model, self.mem = model, pool_tensor
        num_blocks, bs = pool_tensor.shape[2], pool_tensor.shape[4]
        self.handle = C.c_void_p()
        _check(L.q4d_kv_pool_create(model.handle, C.c_int32(num_blocks), C.c_int32(bs), _ptr(pool_tensor),
                                    C.c_size_t(pool_tensor.numel() * 2), C.byref(self.handle)))

    def close(self):
        if self.handle:
            lib().q4d_kv_pool_destroy(self.handle)
            self.handle = C.c_void_p()

    def request_admit(self, rid, prefilled_len):
        _check(lib().q4d_request_admit(self.handle, C.c_int64(rid), C.c_int32(prefilled_len)))

    def request_release(self, rid):
        _check(lib().q4d_request_release(self.handle, C.c_int64(rid)))

    def request_len(self, rid):
        out = C.c_int32()
        _check(lib().q4d_request_len(self.handle, C.c_int64(rid), C.byref(out)))
        return out.value

    def request_count(self):
        out = C.c_int32()
        _check(lib().q4d_request_count(self.handle, C.byref(out)))
        return out.value


def _step_args(ids, block_tables):
    ids = np.ascontiguousarray(ids, dtype=np.int64)
    bt = np.ascontiguousarray(block_tables, dtype=np.int32)
    if bt.ndim != 2 or bt.shape[0] != ids.size:
        raise ValueError("block_tables must be [n][max_blocks]")
    return ids, bt


def decode_step(model, pool, request_ids, last_tokens, block_tables, next_tokens, logits=None, stream=None):
    """q4d_decode_step: host ids / tokens / block tables, device outputs."""
    ids, bt = _step_args(request_ids, block_tables)
    toks = np.ascontiguousarray(last_tokens, dtype=np.int32)
    _check(lib().q4d_decode_step(model.handle, pool.handle, C.c_int32(ids.size), _ptr(ids), _ptr(toks), _ptr(bt),
                                 C.c_int32(bt.shape[1]), _ptr(next_tokens), _ptr(logits), _stream(stream)))


def prefill(model, pool, request_id, tokens, start_pos, block_table, next_token=None, logits=None, stream=None):
    """q4d_prefill: processes tokens[start_pos:] of a prompt into the request's blocks and admits the request."""
    t = np.ascontiguousarray(tokens, dtype=np.int32)
    bt = np.ascontiguousarray(block_table, dtype=np.int32)
    _check(lib().q4d_prefill(model.handle, pool.handle, C.c_int64(int(request_id)), _ptr(t), C.c_int32(t.size),
                             C.c_int32(int(start_pos)), _ptr(bt), C.c_int32(bt.size), _ptr(next_token), _ptr(logits),
                             _stream(stream)))


class SamplingStruct(C.Structure):
    _fields_ = [("temperature", C.c_void_p), ("top_k", C.c_void_p), ("top_p", C.c_void_p), ("u", C.c_void_p)]


def _sampling(temperature, top_k, top_p, u):
    """Host arrays of the per-request settings as a q4d_sampling (the arrays are returned too: keep them alive)."""
    arrs = (np.ascontiguousarray(temperature, dtype=np.float32), np.ascontiguousarray(top_k, dtype=np.int32),
            np.ascontiguousarray(top_p, dtype=np.float32), np.ascontiguousarray(u, dtype=np.float32))
    st = SamplingStruct(*(a.ctypes.data for a in arrs))
    return st, arrs


def decode_step_sampled(model, pool, request_ids, last_tokens, block_tables, temperature, top_k, top_p, u,
                        next_tokens, logits=None, stream=None):
    """q4d_decode_step_sampled: the step, with next_tokens drawn by temperature / top-k / top-p from the given u."""
    ids, bt = _step_args(request_ids, block_tables)
    toks = np.ascontiguousarray(last_tokens, dtype=np.int32)
    st, keep = _sampling(temperature, top_k, top_p, u)
    _check(lib().q4d_decode_step_sampled(model.handle, pool.handle, C.c_int32(ids.size), _ptr(ids), _ptr(toks),
                                         _ptr(bt), C.c_int32(bt.shape[1]), C.byref(st), _ptr(next_tokens),
                                         _ptr(logits), _stream(stream)))
    del keep


def sample(logits, temperature, top_k, top_p, u, stream=None):
    """q4d_sample on a device tensor of logits f32 [n][vocab]; returns the drawn tokens (device int32 [n])."""
    out = torch.empty(logits.shape[0], dtype=torch.int32, device=logits.device)
    st, keep = _sampling(temperature, top_k, top_p, u)
    _check(lib().q4d_sample(_ptr(logits), C.c_int32(logits.shape[0]), C.c_int32(logits.shape[1]), C.byref(st),
                            _ptr(out), _stream(stream)))
    del keep
    return out


def decode_step_chained(model, pool, request_ids, last_tokens_device, block_tables, next_tokens, logits=None,
                        stream=None):
    """q4d_decode_step_chained: the fed-in tokens are a device tensor."""
    ids, bt = _step_args(request_ids, block_tables)
    _check(lib().q4d_decode_step_chained(model.handle, pool.handle, C.c_int32(ids.size), _ptr(ids),
                                         _ptr(last_tokens_device), _ptr(bt), C.c_int32(bt.shape[1]),
                                         _ptr(next_tokens), _ptr(logits), _stream(stream)))


def decode_step_host(model, pool, request_ids, last_tokens, block_tables, want_logits=False, stream=None):
    """q4d_decode_step_host: host inputs and host outputs; returns (next_tokens, logits or None) as numpy."""
    ids, bt = _step_args(request_ids, block_tables)
    toks = np.ascontiguousarray(last_tokens, dtype=np.int32)
    nxt = np.empty(ids.size, dtype=np.int32)
    lg = np.empty((ids.size, model.shape.vocab), dtype=np.float32) if want_logits else None
    _check(lib().q4d_decode_step_host(model.handle, pool.handle, C.c_int32(ids.size), _ptr(ids), _ptr(toks),
                                      _ptr(bt), C.c_int32(bt.shape[1]), _ptr(nxt), _ptr(lg), _stream(stream)))
    return nxt, lg


# --------------------------------------------------------- single operations

_SCRATCH = {}


def op_scratch(device="cuda"):
    """A zero-initialised scratch buffer for the single-operation entry points (one per device)."""
    key = str(torch.device(device))
    if key not in _SCRATCH:
        _SCRATCH[key] = torch.zeros(lib().q4d_op_scratch_bytes(), dtype=torch.uint8, device=device)
    return _SCRATCH[key]


def q4_gemm(w, x, n, prologue=0, epilogue=0, out=None, stream=None):
    """w = (q int32 [N][K/8], scales bf16, biases bf16); x bf16 [n][K] (or [n][2K] with prologue 1)."""
    q = w[0]
    N, K = q.shape[0], q.shape[1] * 8
    qt = _qt(w)
    if out is None:
        out = torch.empty(n, N, dtype=torch.float32 if epilogue == 2 else torch.bfloat16, device=x.device)
    _check(lib().q4d_q4_gemm(C.byref(qt), C.c_int32(N), C.c_int32(K), _ptr(x), C.c_int32(x.stride(0)), C.c_int32(n),
                             C.c_int32(prologue), C.c_int32(epilogue), _ptr(out), C.c_int32(out.stride(0)),
                             _ptr(op_scratch(x.device)), _stream(stream)))
    return out


def q4_gemm_noalloc(w, x, n, out, prologue=0, epilogue=0, stream=None):
    """q4d_q4_gemm_noalloc: like q4_gemm but with the library's built-in scratch; `out` must be preallocated."""
    q = w[0]
    N, K = q.shape[0], q.shape[1] * 8
    qt = _qt(w)
    _check(lib().q4d_q4_gemm_noalloc(C.byref(qt), C.c_int32(N), C.c_int32(K), _ptr(x), C.c_int32(x.stride(0)),
                                     C.c_int32(n), C.c_int32(prologue), C.c_int32(epilogue), _ptr(out),
                                     C.c_int32(out.stride(0)), _stream(stream)))
    return out


def rmsnorm(x, w, eps, stream=None):
    y = torch.empty_like(x)
    _check(lib().q4d_rmsnorm(_ptr(x), _ptr(w), C.c_float(eps), C.c_int32(x.shape[0]), C.c_int32(x.shape[1]), _ptr(y),
                             _stream(stream)))
    return y


def embed(table, tokens, stream=None):
    q = table[0]
    vocab, H = q.shape[0], q.shape[1] * 8
    qt = _qt(table)
    x = torch.empty(tokens.numel(), H, dtype=torch.bfloat16, device=tokens.device)
    _check(lib().q4d_embed(C.byref(qt), C.c_int32(vocab), C.c_int32(H), _ptr(tokens), C.c_int32(tokens.numel()),
                           _ptr(x), _stream(stream)))
    return x


def rope_append(qkv, q_norm, k_norm, eps, rope, nq, nkv, lens, block_tables, pool_k, pool_v, stream=None):
    n = qkv.shape[0]
    q_out = torch.empty(n, nq, 128, dtype=torch.bfloat16, device=qkv.device)
    _check(lib().q4d_rope_append(_ptr(qkv), _ptr(q_norm), _ptr(k_norm), C.c_float(eps), _ptr(rope), C.c_int32(n),
                                 C.c_int32(nq), C.c_int32(nkv), _ptr(lens), _ptr(block_tables),
                                 C.c_int32(block_tables.shape[1]), _ptr(pool_k), _ptr(pool_v), _ptr(q_out),
                                 _stream(stream)))
    return q_out


def paged_attention(q, pool_k, pool_v, lens_host, block_tables_device, chunk_tokens=0, stream=None):
    n, nq = q.shape[0], q.shape[1]
    nkv = pool_k.shape[1]
    lens_host = np.ascontiguousarray(lens_host, dtype=np.int32)
    lens_dev = torch.from_numpy(lens_host).to(q.device)
    out = torch.empty_like(q)
    _check(lib().q4d_paged_attention(_ptr(q), _ptr(pool_k), _ptr(pool_v), C.c_int32(n), C.c_int32(nq), C.c_int32(nkv),
                                     _ptr(lens_host), _ptr(lens_dev), _ptr(block_tables_device),
                                     C.c_int32(block_tables_device.shape[1]), C.c_int32(chunk_tokens), _ptr(out),
                                     _ptr(op_scratch(q.device)), _stream(stream)))
    return out


def argmax(logits, stream=None):
    out = torch.empty(logits.shape[0], dtype=torch.int32, device=logits.device)
    _check(lib().q4d_argmax(_ptr(logits), C.c_int32(logits.shape[0]), C.c_int32(logits.shape[1]), _ptr(out),
                            _stream(stream)))
    return out


def debug_dequant(w, stream=None):
    q = w[0]
    N, K = q.shape[0], q.shape[1] * 8
    qt = _qt(w)
    out = torch.empty(N, K, dtype=torch.float32, device=q.device)
    _check(lib().q4d_debug_dequant(C.byref(qt), C.c_int32(N), C.c_int32(K), _ptr(out), _stream(stream)))
    return out


def debug_kv_gather(pool, layer, block_table_device, length, stream=None):
    nkv = pool.model.shape.n_kv_heads
    k = torch.empty(length, nkv, 128, dtype=torch.bfloat16, device=block_table_device.device)
    v = torch.empty_like(k)
    _check(lib().q4d_debug_kv_gather(pool.handle, C.c_int32(layer), _ptr(block_table_device), C.c_int32(length),
                                     _ptr(k), _ptr(v), _stream(stream)))
    return k, v


def debug_run_layers(model, pool, request_ids, block_tables, layer_begin, layer_end, x_in, stream=None):
    """q4d_debug_run_layers: layers [layer_begin, layer_end) of the production path from the hidden state x_in."""
    ids, bt = _step_args(request_ids, block_tables)
    x_out = torch.empty_like(x_in)
    _check(lib().q4d_debug_run_layers(model.handle, pool.handle, C.c_int32(ids.size), _ptr(ids), _ptr(bt),
                                      C.c_int32(bt.shape[1]), C.c_int32(layer_begin), C.c_int32(layer_end),
                                      _ptr(x_in), _ptr(x_out), _stream(stream)))
    return x_out


# ---- caches of the serving loop (host side) ----------------------------------------------

def sha256(data: bytes) -> bytes:
    out = (C.c_uint8 * 32)()
    _check(lib().q4d_sha256(data, C.c_size_t(len(data)), out))
    return bytes(out)


class PrefixCache:
    """q4d_prefix_cache_*: the text prefix cache of Algorithm 2 over block ids."""

    def __init__(self, capacity_bytes, bytes_per_block):
        self.handle = C.c_void_p()
        _check(lib().q4d_prefix_cache_create(C.c_size_t(capacity_bytes), C.c_size_t(bytes_per_block), C.byref(self.handle)))

    def lookup(self, tokens):
        """(blocks, handles) of the longest cached prefix; the start position is 16 * len(blocks)."""
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        mb = t.size // 16
        blocks, handles, hit = np.zeros(max(mb, 1), dtype=np.int32), np.zeros(max(mb, 1), dtype=np.int32), C.c_int32()
        _check(lib().q4d_prefix_lookup(self.handle, _ptr(t), C.c_int32(t.size), C.c_int32(mb), _ptr(blocks), _ptr(handles),
                                       C.byref(hit)))
        return blocks[:hit.value].tolist(), handles[:hit.value].tolist()

    def insert(self, tokens, block_table):
        """(handles, adopted) for the full blocks of the prompt."""
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        bt = np.ascontiguousarray(block_table, dtype=np.int32)
        nb = min(t.size // 16, bt.size)
        handles, adopted = np.zeros(max(nb, 1), dtype=np.int32), np.zeros(max(nb, 1), dtype=np.int32)
        _check(lib().q4d_prefix_insert(self.handle, _ptr(t), C.c_int32(t.size), _ptr(bt), C.c_int32(nb), _ptr(handles),
                                       _ptr(adopted)))
        return handles[:nb].tolist(), adopted[:nb].tolist()

    def release(self, handles):
        h = np.ascontiguousarray(handles, dtype=np.int32)
        _check(lib().q4d_prefix_release(self.handle, _ptr(h), C.c_int32(h.size)))

    def evict(self, bytes_to_free=0, max_out=1 << 16):
        out, n = np.zeros(max_out, dtype=np.int32), C.c_int32()
        _check(lib().q4d_prefix_evict(self.handle, C.c_size_t(bytes_to_free), C.c_int32(max_out), _ptr(out), C.byref(n)))
        return out[:n.value].tolist()

    def stats(self):
        v = [C.c_int64() for _ in range(4)]
        _check(lib().q4d_prefix_cache_stats(self.handle, *(C.byref(x) for x in v)))
        return dict(zip(("entries", "bytes", "lookups", "hit_blocks"), (x.value for x in v)))

    def close(self):
        if self.handle:
            lib().q4d_prefix_cache_destroy(self.handle)
            self.handle = C.c_void_p()


class ContentEntry(C.Structure):
    _fields_ = [("hash", C.c_uint8 * 32), ("embeddings", C.c_void_p), ("bytes", C.c_int64), ("n_tokens", C.c_int32),
                ("n_blocks", C.c_int32)]


class ContentCache:
    """q4d_content_cache_*: the content-hash store of Algorithm 3 (embeddings handle + KV blocks per image hash)."""

    def __init__(self, capacity_bytes, max_blocks=4096):
        self.handle = C.c_void_p()
        self.max_blocks = max_blocks
        _check(lib().q4d_content_cache_create(C.c_size_t(capacity_bytes), C.byref(self.handle)))

    def lookup(self, pixels: bytes):
        """(hit, entry, blocks): on a miss the entry carries only the hash."""
        e, hit = ContentEntry(), C.c_int32()
        blocks = np.zeros(self.max_blocks, dtype=np.int32)
        _check(lib().q4d_content_lookup(self.handle, pixels, C.c_size_t(len(pixels)), C.byref(e), C.c_int32(self.max_blocks),
                                        _ptr(blocks), C.byref(hit)))
        return bool(hit.value), e, blocks[:e.n_blocks].tolist() if hit.value else []

    def store(self, entry, blocks):
        b = np.ascontiguousarray(blocks, dtype=np.int32)
        entry.n_blocks = b.size
        _check(lib().q4d_content_store(self.handle, C.byref(entry), _ptr(b)))

    def release(self, hash32: bytes):
        _check(lib().q4d_content_release(self.handle, (C.c_uint8 * 32).from_buffer_copy(hash32)))

    def evict(self, bytes_to_free=0):
        """Evicted (entry, blocks) pairs, least recently used first, until the store is within its budget."""
        gone = []
        while True:
            e, did = ContentEntry(), C.c_int32()
            blocks = np.zeros(self.max_blocks, dtype=np.int32)
            _check(lib().q4d_content_evict(self.handle, C.c_size_t(bytes_to_free), C.byref(e), C.c_int32(self.max_blocks),
                                           _ptr(blocks), C.byref(did)))
            if not did.value:
                return gone
            gone.append((e, blocks[:e.n_blocks].tolist()))
            bytes_to_free = max(0, bytes_to_free - e.bytes)

    def stats(self):
        n, b = C.c_int64(), C.c_int64()
        _check(lib().q4d_content_cache_stats(self.handle, C.byref(n), C.byref(b)))
        return {"entries": n.value, "bytes": b.value}

    def close(self):
        if self.handle:
            lib().q4d_content_cache_destroy(self.handle)
            self.handle = C.c_void_p()
