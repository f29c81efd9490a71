"""Helpers shared by the GPU parity tests (comparison utilities and scenario setup)."""
import numpy as np
import torch

from oracle import q4d_oracle as orc
from workload import gen


def bits(t):
    """torch bf16 tensor -> numpy uint16 bit patterns (host)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def from_bits(a, device="cuda"):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).to(device)


def bf16_ulp_distance(a_bits, b_bits):
    """Distance in bf16 steps between two arrays of bf16 bit patterns (sign-magnitude aware)."""
    def key(b):
        b = b.astype(np.int64)
        return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)
    return np.abs(key(np.asarray(a_bits)) - key(np.asarray(b_bits)))


def assert_bf16_close(got_bits, want_bits, max_ulp=1, max_mismatch_frac=0.01, what="", floor_frac=0.25):
    """Every element within max_ulp bf16 steps of the expected value, where the step is that of the expected
    element or, for elements that are small because their sum cancelled, that of floor_frac * rms of the tensor;
    and at most max_mismatch_frac of the elements different at all.

    Both sides round a value computed in different precision (fp32 on the GPU, fp64 in the oracle) to bf16,
    so a small fraction of elements that sit next to a rounding boundary land one step apart.
    """
    got, want = _f64(got_bits), _f64(want_bits)
    rms = float(np.sqrt((want ** 2).mean())) if want.size else 0.0
    step = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(want), max(floor_frac * rms, 1e-30)))) - 7)
    worst = float((np.abs(got - want) / step).max(initial=0.0))
    frac = float((np.asarray(got_bits) != np.asarray(want_bits)).mean()) if want.size else 0.0
    assert worst <= max_ulp, f"{what}: {worst:.2f} bf16 steps off (> {max_ulp})"
    assert frac <= max_mismatch_frac, f"{what}: {frac:.4%} of elements differ (> {max_mismatch_frac:.2%})"
    return frac


def _f64(b):
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


class Scenario:
    """Weights, pool and requests on the GPU, mirrored on the host for the oracle."""

    def __init__(self, shape, lens, seed=0, extra_blocks=8, device="cuda"):
        self.shape, self.device = shape, device
        self.weights = gen.make_weights(shape, seed, device)
        need = sum((l + 1 + 64 + 15) // 16 for l in lens) + extra_blocks
        self.pool = gen.make_pool(shape, need, device)
        self.alloc = gen.BlockAllocator(need, seed)
        self.lens = list(lens)
        self.blocks = []
        for r, l in enumerate(lens):
            blk = self.alloc.alloc((l + 1 + 15) // 16)
            gen.fill_blocks(self.pool, blk, seed, "kv", r)
            self.blocks.append(blk)
        rng = np.random.default_rng(seed + 1000)
        self.tokens = rng.integers(0, shape.vocab, size=len(lens)).astype(np.int32)
        self.oracle = orc.OracleModel(shape, self.weights)
        self.host_pool = orc.to_np(self.pool).copy()

    def block_tables(self):
        for r, l in enumerate(self.lens):
            need = (l + 1 + 15) // 16
            if need > len(self.blocks[r]):
                self.blocks[r].extend(self.alloc.alloc(need - len(self.blocks[r])))
        mb = max(len(b) for b in self.blocks)
        bt = np.zeros((len(self.lens), mb), dtype=np.int32)
        for r, b in enumerate(self.blocks):
            bt[r, :len(b)] = b
        return bt


def rel_err(got_bits, want_bits):
    """(max |got - want| / rms(want), rms(got - want) / rms(want), fraction of differing elements)."""
    g, w = orc.bf16_to_f64(got_bits), orc.bf16_to_f64(want_bits)
    rms = float(np.sqrt((w ** 2).mean())) or 1.0
    d = g - w
    return float(np.abs(d).max()) / rms, float(np.sqrt((d ** 2).mean())) / rms, float((got_bits != want_bits).mean())


def gpu_layer(q4d, shape, weights, layer, x, pool_t, lens, dlens, dbt, oracle_pool=None, bt=None):
    """One decoder layer on the GPU, composed from the library's single-operation entry points (the same
    kernels the step driver launches).  x (bf16 [n][H]) is updated in place.  If oracle_pool is given, the
    K, V the layer appended are replaced by the oracle's before attention reads them (teacher forcing)."""
    lw = weights["layers"][layer]
    n = x.shape[0]
    y = q4d.rmsnorm(x, lw["attn_norm"], shape.rms_eps)
    qkv = q4d.q4_gemm(lw["wqkv"], y, n, epilogue=0)
    q = q4d.rope_append(qkv, lw.get("q_norm"), lw.get("k_norm"), shape.rms_eps, weights["rope"], shape.n_q_heads,
                        shape.n_kv_heads, dlens, dbt, pool_t[layer, 0], pool_t[layer, 1])
    if oracle_pool is not None:
        for r, l in enumerate(lens):
            blk, slot = int(bt[r, l // 16]), l % 16
            pool_t[layer, :, blk, :, slot] = from_bits(oracle_pool[layer, :, blk, :, slot])
    att = q4d.paged_attention(q, pool_t[layer, 0], pool_t[layer, 1], lens, dbt)
    q4d.q4_gemm(lw["wo"], att.view(n, -1), n, epilogue=1, out=x)
    y = q4d.rmsnorm(x, lw["mlp_norm"], shape.rms_eps)
    gu = q4d.q4_gemm(lw["w_gate_up"], y, n, epilogue=0)
    q4d.q4_gemm(lw["w_down"], gu, n, prologue=1, epilogue=1, out=x)
    return x
